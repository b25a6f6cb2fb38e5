// Pipelined tile kernels: the bandwidth path of all four S2A entry points.
//
// A persistent CTA walks tiles of `tile_rows` consecutive rows.  One extra warp moves
// whole tiles between HBM and shared memory with bulk asynchronous copies (the TMA
// engine, no multicast): loads complete on a "full" mbarrier per stage, the consumer
// warps rewrite the tile in place in shared memory (x -> y, grad_out -> grad_in) and
// produce or consume the packed codes and the per-row (min, s), signal a "done"
// mbarrier, and the copy warp streams the results back out and refills the stage.
// Memory-level parallelism therefore comes from the copy engine, not from registers or
// occupancy, and rows of any alignment are handled because a tile always starts and
// ends on a multiple of 32 elements (16-byte aligned data AND code bytes).
//
// Inside a tile a "unit" of 8, 16, 32 or 128 lanes owns one row at a time and keeps it
// in registers; row reductions are warp shuffles (plus one shared-memory hop for
// 128-lane units).  Rows are read as 16-byte vectors when row_len allows it and
// otherwise as 2-element words on the tile's even-element grid, where a row of odd
// length shares its first or last word (and code byte) with its neighbour: the two rows
// of such a pair are handled back to back by the same unit.
//
// Every wait on an mbarrier is bounded; a wait that runs out sets a bit in the
// per-device error word and the CTA winds down.
#pragma once
#include "s2a_common.cuh"
#include "s2a_launch.h"

#include <atomic>
#include <type_traits>

namespace s2a {
namespace {

constexpr uint32_t kSpinLimit = 1u << 22;
constexpr uint32_t kSuspendNs = 100000;             // longest sleep inside one try
constexpr uint64_t kWaitLimitNs = 2000000000ull;   // 2 s: a wait this long has failed
constexpr int kMaxStages = 8;
constexpr int kHeaderBytes = 4096;  // barriers, reduction scratch, derivative tables
constexpr int kRedOffset = 256;     // float[2 slots][16 units][4 warps]  (multi-warp units)
constexpr int kFlagOffset = 768;    // int[16]: abort flag per multi-warp unit
constexpr int kTabOffset = 1024;    // float[units][16]: Eq. 12 table per unit (<= 32 units)

enum { kVec16 = 0, kPair = 1 };

struct TileKernelArgs {
  const unsigned char* in;
  unsigned char* out;
  unsigned char* codes;
  unsigned char* meta;
  uint64_t tiles_per_cta;  // n_tiles / grid; the first tiles_extra CTAs take one more
  uint32_t tiles_extra;    // n_tiles % grid
  uint32_t row_len;
  uint32_t tile_rows;
  uint32_t data_bytes;   // per tile
  uint32_t code_bytes;   // per tile
  uint32_t meta_bytes;   // per tile
  uint32_t code_off;     // offsets inside a stage
  uint32_t meta_off;
  uint32_t stage_bytes;
  uint32_t stages;
  uint32_t spread_units;     // 1: sub-warp units of a warp take groups a fixed stride apart
  uint32_t tab_off;          // byte offset of the wide derivative tables (8-bit codes), else 0
  uint32_t prefetch_tiles;   // tiles whose inputs the copy lane asks into the L2 before the dependency wait
  uint32_t prefetch_ahead;   // steady state: with the load of tile i, tile i + this many is asked into the L2 (0: off)
  uint32_t ragged_codes;     // 1: a tile's code bytes start anywhere (tile_kernel<WORK, true> only), see there
  unsigned int* error_word;  // device address of the per-device error word
};

// ---------------------------------------------------------------- PTX wrappers
__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return (uint32_t)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)),
               "r"(bytes)
               : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}
// The same test, but the warp may sleep in hardware for up to `ns` nanoseconds and is woken
// when the phase completes: a waiting warp then takes no issue slots from the warps it is
// waiting for (a polling loop of the copy lane was a fifth of all instructions issued).
__device__ __forceinline__ bool mbar_try_wait_suspend(uint64_t* bar, uint32_t parity, uint32_t ns) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity), "r"(ns)
      : "memory");
  return ok != 0;
}
__device__ __forceinline__ uint64_t global_timer_ns() {
  uint64_t t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
// Bounded wait for the phase with the given parity to complete: gives up after
// kWaitLimitNs of wall time or kSpinLimit tries, whichever comes first, and records why.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, unsigned int* err, unsigned err_bit,
                                          uint64_t limit_ns = kWaitLimitNs) {
  if (mbar_try_wait(bar, parity)) return true;
  const uint64_t t0 = global_timer_ns();
#pragma unroll 1
  for (uint32_t i = 0; i < kSpinLimit; ++i) {
    if (mbar_try_wait_suspend(bar, parity, kSuspendNs)) return true;
    if (global_timer_ns() - t0 > limit_ns) break;
  }
  atomicOr(err, err_bit);
  return false;
}
__device__ __forceinline__ void fence_barrier_init() {
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void fence_proxy_async() {
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}
// global -> shared bulk copy; completion is counted in bytes on `bar`.
__device__ __forceinline__ void bulk_load(void* dst_smem, const void* src, uint32_t bytes,
                                          uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::
          "r"(smem_u32(dst_smem)),
      "l"(src), "r"(bytes), "r"(smem_u32(bar))
      : "memory");
}
// Asks for a span of this GPU's global memory to be brought into the L2.  A prefetch changes
// no architectural state (the L2 is the point of coherence: a line written later by an
// earlier kernel is simply updated there), so it may run ahead of the dependency wait.
__device__ __forceinline__ void bulk_prefetch_l2(const void* src, uint32_t bytes) {
  asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(src), "r"(bytes) : "memory");
}
// shared -> global bulk copy, tracked by the thread's bulk-group.
__device__ __forceinline__ void bulk_store(void* dst, const void* src_smem, uint32_t bytes) {
  asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(dst),
               "r"(smem_u32(src_smem)), "r"(bytes)
               : "memory");
}
__device__ __forceinline__ void bulk_commit() {
  asm volatile("cp.async.bulk.commit_group;" ::: "memory");
}
template <int N>
__device__ __forceinline__ void bulk_wait_read() {
  asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory");
}
__device__ __forceinline__ void bulk_wait_all() {
  asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
}
// Programmatic dependent launch: the next kernel of the stream may be scheduled while
// this one drains, and parks at grid_dependency_wait() until this one has completed and
// its writes are visible.  Both are no-ops for a kernel launched without the attribute.
__device__ __forceinline__ void grid_launch_dependents() {
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}
__device__ __forceinline__ void grid_dependency_wait() {
  asm volatile("griddepcontrol.wait;" ::: "memory");
}
__device__ __forceinline__ void named_bar_sync(int id, int threads) {
  asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(threads) : "memory");
}

// ---------------------------------------------------------------- shared-memory access
// One "access" is what a lane reads or writes at a time: EPA elements and the code
// bytes that belong to them.
template <int DT, int VMODE> struct Acc;

template <> struct Acc<kBF16, kVec16> {
  static constexpr int EPA = 8;
  using Raw = uint4;
  static __device__ __forceinline__ Raw load(const unsigned char* d, uint32_t a) {
    return *(const uint4*)(d + (size_t)a * 16);
  }
  static __device__ __forceinline__ void widen(const Raw& r, float* v) {
    const uint32_t w[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      v[2 * k] = __uint_as_float(w[k] << 16);
      v[2 * k + 1] = __uint_as_float(w[k] & 0xffff0000u);
    }
  }
  // Rounds to the I/O type, stores, and leaves in v the values as written.
  static __device__ __forceinline__ void narrow_store(unsigned char* d, uint32_t a, float* v, int) {
    uint32_t w[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      __nv_bfloat162 b = __floats2bfloat162_rn(v[2 * k], v[2 * k + 1]);
      w[k] = *(uint32_t*)&b;
      v[2 * k] = __uint_as_float(w[k] << 16);
      v[2 * k + 1] = __uint_as_float(w[k] & 0xffff0000u);
    }
    *(uint4*)(d + (size_t)a * 16) = make_uint4(w[0], w[1], w[2], w[3]);
  }
  static __device__ __forceinline__ uint32_t load_codes(const unsigned char* c, uint32_t a) {
    return *(const uint32_t*)(c + (size_t)a * 4);
  }
  static __device__ __forceinline__ void store_codes(unsigned char* c, uint32_t a, uint32_t bits) {
    *(uint32_t*)(c + (size_t)a * 4) = bits;
  }
};

template <> struct Acc<kF32, kVec16> {
  static constexpr int EPA = 4;
  using Raw = float4;
  static __device__ __forceinline__ Raw load(const unsigned char* d, uint32_t a) {
    return *(const float4*)(d + (size_t)a * 16);
  }
  static __device__ __forceinline__ void widen(const Raw& r, float* v) {
    v[0] = r.x; v[1] = r.y; v[2] = r.z; v[3] = r.w;
  }
  static __device__ __forceinline__ void narrow_store(unsigned char* d, uint32_t a, float* v, int) {
    *(float4*)(d + (size_t)a * 16) = make_float4(v[0], v[1], v[2], v[3]);
  }
  static __device__ __forceinline__ uint32_t load_codes(const unsigned char* c, uint32_t a) {
    return *(const uint16_t*)(c + (size_t)a * 2);
  }
  static __device__ __forceinline__ void store_codes(unsigned char* c, uint32_t a, uint32_t bits) {
    *(uint16_t*)(c + (size_t)a * 2) = (uint16_t)bits;
  }
};

// Pair mode: `keep` says which of the two elements belong to the row (bit 0: low,
// bit 1: high); the other half of a shared word is left untouched.
template <> struct Acc<kBF16, kPair> {
  static constexpr int EPA = 2;
  using Raw = uint32_t;
  static __device__ __forceinline__ Raw load(const unsigned char* d, uint32_t a) {
    return *(const uint32_t*)(d + (size_t)a * 4);
  }
  static __device__ __forceinline__ void widen(const Raw& r, float* v) {
    v[0] = __uint_as_float(r << 16);
    v[1] = __uint_as_float(r & 0xffff0000u);
  }
  static __device__ __forceinline__ void narrow_store(unsigned char* d, uint32_t a, float* v, int keep) {
    __nv_bfloat162 b = __floats2bfloat162_rn(v[0], v[1]);
    uint32_t w = *(uint32_t*)&b;
    v[0] = __uint_as_float(w << 16);
    v[1] = __uint_as_float(w & 0xffff0000u);
    if (keep == 3) *(uint32_t*)(d + (size_t)a * 4) = w;
    else if (keep == 1) *(uint16_t*)(d + (size_t)a * 4) = (uint16_t)w;
    else if (keep == 2) *(uint16_t*)(d + (size_t)a * 4 + 2) = (uint16_t)(w >> 16);
  }
  static __device__ __forceinline__ uint32_t load_codes(const unsigned char* c, uint32_t a) {
    return c[a];
  }
  static __device__ __forceinline__ void store_codes(unsigned char* c, uint32_t a, uint32_t bits) {
    c[a] = (unsigned char)bits;
  }
};

template <> struct Acc<kF32, kPair> {
  static constexpr int EPA = 2;
  using Raw = float2;
  static __device__ __forceinline__ Raw load(const unsigned char* d, uint32_t a) {
    return *(const float2*)(d + (size_t)a * 8);
  }
  static __device__ __forceinline__ void widen(const Raw& r, float* v) {
    v[0] = r.x; v[1] = r.y;
  }
  static __device__ __forceinline__ void narrow_store(unsigned char* d, uint32_t a, float* v, int keep) {
    if (keep == 3) *(float2*)(d + (size_t)a * 8) = make_float2(v[0], v[1]);
    else if (keep == 1) *(float*)(d + (size_t)a * 8) = v[0];
    else if (keep == 2) *(float*)(d + (size_t)a * 8 + 4) = v[1];
  }
  static __device__ __forceinline__ uint32_t load_codes(const unsigned char* c, uint32_t a) {
    return c[a];
  }
  static __device__ __forceinline__ void store_codes(unsigned char* c, uint32_t a, uint32_t bits) {
    c[a] = (unsigned char)bits;
  }
};

// ---------------------------------------------------------------- units
enum { kOpMax = 0, kOpMin = 1, kOpSum = 2 };

template <int OP>
__device__ __forceinline__ float op2(float a, float b) {
  return OP == kOpMax ? fmaxf(a, b) : (OP == kOpMin ? fminf(a, b) : a + b);
}

template <int UNIT>
struct Unit {
  int ul;       // lane within the unit
  int uid;      // unit within the CTA
  float* red;   // reduction scratch of this unit (multi-warp units only)
  int phase;

  template <int OP>
  __device__ __forceinline__ float reduce(float v) {
    constexpr int W = UNIT < 32 ? UNIT : 32;
#pragma unroll
    for (int o = W / 2; o > 0; o >>= 1) v = op2<OP>(v, __shfl_xor_sync(0xffffffffu, v, o));
    if (UNIT > 32) {
      constexpr int NW = UNIT / 32;
      float* slot = red + (phase & 1) * 64;
      if ((ul & 31) == 0) slot[ul >> 5] = v;
      named_bar_sync(1 + uid, UNIT);
      v = slot[0];
#pragma unroll
      for (int k = 1; k < NW; ++k) v = op2<OP>(v, slot[k]);
      ++phase;
    }
    return v;
  }
  // Minimum of a packed bfloat16x2 over the unit, both halves at once (a row's minimum and the
  // negative of its maximum travel together: one shuffle sequence, one exchange between warps).
  __device__ __forceinline__ uint32_t reduce_min_bf16x2(uint32_t w) {
    constexpr int W = UNIT < 32 ? UNIT : 32;
#pragma unroll
    for (int o = W / 2; o > 0; o >>= 1) {
      const uint32_t other = __shfl_xor_sync(0xffffffffu, w, o);
      const __nv_bfloat162 r = __hmin2(*(const __nv_bfloat162*)&w, *(const __nv_bfloat162*)&other);
      w = *(const uint32_t*)&r;
    }
    if (UNIT > 32) {
      constexpr int NW = UNIT / 32;
      uint32_t* slot = (uint32_t*)red + (phase & 1) * 64;
      if ((ul & 31) == 0) slot[ul >> 5] = w;
      named_bar_sync(1 + uid, UNIT);
      w = slot[0];
#pragma unroll
      for (int k = 1; k < NW; ++k) {
        const uint32_t other = slot[k];
        const __nv_bfloat162 r = __hmin2(*(const __nv_bfloat162*)&w, *(const __nv_bfloat162*)&other);
        w = *(const uint32_t*)&r;
      }
      ++phase;
    }
    return w;
  }
  // Orders shared-memory accesses of the unit's lanes (and keeps them in step).
  __device__ __forceinline__ void sync() {
    if (UNIT > 32) named_bar_sync(1 + uid, UNIT);
    else __syncwarp();
  }
};

// Row minimum and maximum of bfloat16-valued numbers in ONE shuffle sequence: the pair
// (min, -max) travels as a packed bfloat16x2 and is folded with a packed minimum (negation
// is exact).  Sub-warp and warp units only.
template <int UNIT>
__device__ __forceinline__ void reduce_minmax_bf16(float& mn, float& mx) {
  static_assert(UNIT <= 32, "warp-level reduction");
  __nv_bfloat162 p = __floats2bfloat162_rn(mn, -mx);  // exact: both are bfloat16 values (or +-inf)
  uint32_t w = *(uint32_t*)&p;
#pragma unroll
  for (int o = UNIT / 2; o > 0; o >>= 1) {
    uint32_t other = __shfl_xor_sync(0xffffffffu, w, o);
    __nv_bfloat162 r = __hmin2(*(__nv_bfloat162*)&w, *(__nv_bfloat162*)&other);
    w = *(uint32_t*)&r;
  }
  mn = __uint_as_float(w << 16);
  mx = -__uint_as_float(w & 0xffff0000u);
}

// Geometry of one row inside a tile, in accesses.
struct RowGeom {
  uint32_t a0;    // first access (tile-relative)
  uint32_t n_acc; // accesses covering the row
  bool head;      // pair mode: low element of the first access belongs to the previous row
  bool tail;      // pair mode: high element of the last access belongs to the next row
};

template <int DT, int VMODE>
__device__ __forceinline__ RowGeom row_geom(uint32_t r, uint32_t L) {
  RowGeom g;
  if (VMODE == kVec16) {
    constexpr int EPA = Acc<DT, VMODE>::EPA;
    g.n_acc = L / EPA;
    g.a0 = r * g.n_acc;
    g.head = false;
    g.tail = false;
  } else {
    uint32_t e0 = r * L;
    g.a0 = e0 >> 1;
    g.n_acc = ((e0 + L - 1) >> 1) - g.a0 + 1;
    g.head = (e0 & 1u) != 0;
    g.tail = ((e0 + L) & 1u) != 0;
  }
  return g;
}

// e^d for d = x - max <= 0.  One multiply and the hardware 2^x (2 ulp): the rounding of the
// product moves the result by at most 2^-24 |d| relative, which is the allowance the softmax
// output carries for the rounding of its exponent's argument.
template <int DT>
__device__ __forceinline__ float exp_eval(float d) {
  return ex2_approx(1.4426950408889634f * d);
}

// ---------------------------------------------------------------- per-row work
// All lanes of a unit call these together.  `active` is false for a unit that has no
// row in this round; it still takes part in the reductions.
template <int KERNEL, int DT, int VMODE, int UNIT, int ITERS>
struct RowWork {
  using A = Acc<DT, VMODE>;
  static constexpr int EPA = A::EPA;

  // Which elements of access i belong to the row (bit k = element k); 0 if none.
  static __device__ __forceinline__ uint32_t keep_mask(const RowGeom& g, uint32_t idx, bool active) {
    if (!active || idx >= g.n_acc) return 0u;
    uint32_t m = (1u << EPA) - 1u;
    if (VMODE == kPair) {
      if (g.head && idx == 0) m &= ~1u;
      if (g.tail && idx == g.n_acc - 1) m &= ~2u;
    }
    return m;
  }

  static __device__ __forceinline__ void gelu_fwd(Unit<UNIT>& u, unsigned char* data, unsigned char* codes,
                                                  float* meta_s, uint32_t r, uint32_t L, bool active) {
    const RowGeom g = row_geom<DT, VMODE>(r, L);
    typename A::Raw raw[ITERS];
    float mn = INFINITY, mx = -INFINITY;
#pragma unroll
    for (int i = 0; i < ITERS; ++i) {
      const uint32_t idx = u.ul + UNIT * i;
      const uint32_t keep = keep_mask(g, idx, active);
      if (keep) {
        raw[i] = A::load(data, g.a0 + idx);
        float v[EPA];
        A::widen(raw[i], v);
#pragma unroll
        for (int k = 0; k < EPA; ++k)
          if (keep >> k & 1) { mn = fminf(mn, v[k]); mx = fmaxf(mx, v[k]); }
      }
    }
    mn = u.template reduce<kOpMin>(mn);
    mx = u.template reduce<kOpMax>(mx);
    const QRange q = make_qrange(fminf(fmaxf(mn, -kClip), kClip), fminf(fmaxf(mx, -kClip), kClip));
    if (active && u.ul == 0) { meta_s[2 * r] = q.mn; meta_s[2 * r + 1] = q.s; }
#pragma unroll
    for (int i = 0; i < ITERS; ++i) {
      const uint32_t idx = u.ul + UNIT * i;
      const uint32_t keep = keep_mask(g, idx, active);
      if (keep) {
        float v[EPA];
        A::widen(raw[i], v);
        uint32_t bits = 0;
#pragma unroll
        for (int k = 0; k < EPA; ++k) {
          if (keep >> k & 1) bits |= quant_code(fminf(fmaxf(v[k], -kClip), kClip), q) << (4 * k);
          v[k] = gelu_eval<DT>(v[k]);
        }
        if (VMODE == kPair && !(keep & 1)) bits |= A::load_codes(codes, g.a0 + idx) & 0xFu;
        A::narrow_store(data, g.a0 + idx, v, (int)keep);
        A::store_codes(codes, g.a0 + idx, bits);
      }
    }
  }

  static __device__ __forceinline__ void softmax_fwd(Unit<UNIT>& u, unsigned char* data, unsigned char* codes,
                                                     float* meta_s, uint32_t r, uint32_t L, bool active) {
    const RowGeom g = row_geom<DT, VMODE>(r, L);
    float e[ITERS][EPA];
    float m = -INFINITY;
#pragma unroll
    for (int i = 0; i < ITERS; ++i) {
      const uint32_t idx = u.ul + UNIT * i;
      const uint32_t keep = keep_mask(g, idx, active);
#pragma unroll
      for (int k = 0; k < EPA; ++k) e[i][k] = -INFINITY;
      if (keep) {
        float v[EPA];
        A::widen(A::load(data, g.a0 + idx), v);
#pragma unroll
        for (int k = 0; k < EPA; ++k)
          if (keep >> k & 1) { e[i][k] = v[k]; m = fmaxf(m, v[k]); }
      }
    }
    m = u.template reduce<kOpMax>(m);
    if (!active) m = 0.0f;
    float z = 0.0f;
#pragma unroll
    for (int i = 0; i < ITERS; ++i)
#pragma unroll
      for (int k = 0; k < EPA; ++k) {
        e[i][k] = exp_eval<DT>(e[i][k] - m);  // elements outside the row: exp(-inf) = 0
        z += e[i][k];
      }
    z = u.template reduce<kOpSum>(z);
    const float rz = __fdiv_rn(1.0f, active ? z : 1.0f);
    float mn = INFINITY, mx = -INFINITY;
#pragma unroll
    for (int i = 0; i < ITERS; ++i) {
      const uint32_t idx = u.ul + UNIT * i;
      const uint32_t keep = keep_mask(g, idx, active);
      if (keep) {
#pragma unroll
        for (int k = 0; k < EPA; ++k) e[i][k] *= rz;
        A::narrow_store(data, g.a0 + idx, e[i], (int)keep);  // e now holds y as written
#pragma unroll
        for (int k = 0; k < EPA; ++k)
          if (keep >> k & 1) { mn = fminf(mn, e[i][k]); mx = fmaxf(mx, e[i][k]); }
      }
    }
    mn = u.template reduce<kOpMin>(mn);
    mx = u.template reduce<kOpMax>(mx);
    const QRange q = make_qrange(mn, mx);
    if (active && u.ul == 0) { meta_s[2 * r] = q.mn; meta_s[2 * r + 1] = q.s; }
#pragma unroll
    for (int i = 0; i < ITERS; ++i) {
      const uint32_t idx = u.ul + UNIT * i;
      const uint32_t keep = keep_mask(g, idx, active);
      if (keep) {
        uint32_t bits = 0;
#pragma unroll
        for (int k = 0; k < EPA; ++k)
          if (keep >> k & 1) bits |= quant_code(e[i][k], q) << (4 * k);
        if (VMODE == kPair && !(keep & 1)) bits |= A::load_codes(codes, g.a0 + idx) & 0xFu;
        A::store_codes(codes, g.a0 + idx, bits);
      }
    }
  }

  static __device__ __forceinline__ void gelu_bwd(Unit<UNIT>& u, unsigned char* data, const unsigned char* codes,
                                                  const float* meta_s, float* tab, float& tab_mn, float& tab_s,
                                                  uint32_t r, uint32_t L, bool active) {
    const RowGeom g = row_geom<DT, VMODE>(r, L);
    const float mn = active ? meta_s[2 * r] : tab_mn;
    const float s = active ? meta_s[2 * r + 1] : tab_s;
    // The 16 values of Eq. 12 this row can take, in binary64; kept while (min, s) repeat.
    if (mn != tab_mn || s != tab_s) {
#pragma unroll
      for (int c = 0; c < 16; c += (UNIT < 16 ? UNIT : 16)) {
        const int code = c + u.ul;
        if (u.ul < 16 && code < 16) tab[code] = (float)gelu_sine_derivative((uint32_t)code, mn, s);
      }
      tab_mn = mn;
      tab_s = s;
    }
    u.sync();
#pragma unroll
    for (int i = 0; i < ITERS; ++i) {
      const uint32_t idx = u.ul + UNIT * i;
      const uint32_t keep = keep_mask(g, idx, active);
      if (keep) {
        float v[EPA];
        A::widen(A::load(data, g.a0 + idx), v);
        const uint32_t bits = A::load_codes(codes, g.a0 + idx);
#pragma unroll
        for (int k = 0; k < EPA; ++k) v[k] *= tab[(bits >> (4 * k)) & 0xFu];
        A::narrow_store(data, g.a0 + idx, v, (int)keep);
      }
    }
  }

  static __device__ __forceinline__ void softmax_bwd(Unit<UNIT>& u, unsigned char* data, const unsigned char* codes,
                                                     const float* meta_s, uint32_t r, uint32_t L, bool active) {
    const RowGeom g = row_geom<DT, VMODE>(r, L);
    const float mn = active ? meta_s[2 * r] : 0.0f;
    const float s = active ? meta_s[2 * r + 1] : 0.0f;
    float gv[ITERS][EPA], yh[ITERS][EPA];
    float dot = 0.0f;
#pragma unroll
    for (int i = 0; i < ITERS; ++i) {
      const uint32_t idx = u.ul + UNIT * i;
      const uint32_t keep = keep_mask(g, idx, active);
      if (keep) {
        A::widen(A::load(data, g.a0 + idx), gv[i]);
        const uint32_t bits = A::load_codes(codes, g.a0 + idx);
#pragma unroll
        for (int k = 0; k < EPA; ++k) {
          yh[i][k] = dequant((bits >> (4 * k)) & 0xFu, mn, s);
          if (keep >> k & 1) dot = fmaf(gv[i][k], yh[i][k], dot);
        }
      }
    }
    dot = u.template reduce<kOpSum>(dot);
#pragma unroll
    for (int i = 0; i < ITERS; ++i) {
      const uint32_t idx = u.ul + UNIT * i;
      const uint32_t keep = keep_mask(g, idx, active);
      if (keep) {
        float v[EPA];
#pragma unroll
        for (int k = 0; k < EPA; ++k) v[k] = yh[i][k] * (gv[i][k] - dot);
        A::narrow_store(data, g.a0 + idx, v, (int)keep);
      }
    }
  }
};

// ---------------------------------------------------------------- work policies
// A policy tells the pipeline skeleton how the consumer lanes of a CTA turn one tile
// in shared memory into its results.  `group` is called by all lanes of a unit for one
// group of consecutive rows (one row, or the two rows of an odd-length pair).
struct StagePtrs {
  unsigned char* data;
  unsigned char* codes;
  float* meta;
};

// Policy 0: the general register-resident form (any row length that fits ITERS).
template <int KERNEL, int DT, int VMODE, int UNIT_, int ITERS>
struct GenericWork {
  static constexpr int kKernel = KERNEL;
  static constexpr int kMaxRegs = 128;
  static constexpr int UNIT = UNIT_;
  using W = RowWork<KERNEL, DT, VMODE, UNIT_, ITERS>;
  struct State {
    float tab_mn, tab_s;
  };
  static __device__ __forceinline__ void init(State& st) {
    st.tab_mn = __int_as_float(0x7fc00000);  // NaN: nothing cached yet
    st.tab_s = st.tab_mn;
  }
  static __device__ __forceinline__ uint32_t rows_per_group(uint32_t L) {
    return (VMODE == kPair && (L & 1u)) ? 2u : 1u;
  }
  static __device__ __forceinline__ void group(Unit<UNIT_>& u, State& st, const StagePtrs& p, float* tab,
                                               uint32_t grp, bool active, uint32_t L) {
    const uint32_t G = rows_per_group(L);
    for (uint32_t h = 0; h < G; ++h) {
      const uint32_t r = active ? grp * G + h : 0;
      if (KERNEL == kGeluFwd) W::gelu_fwd(u, p.data, p.codes, p.meta, r, L, active);
      if (KERNEL == kSoftmaxFwd) W::softmax_fwd(u, p.data, p.codes, p.meta, r, L, active);
      if (KERNEL == kGeluBwd) W::gelu_bwd(u, p.data, p.codes, p.meta, tab, st.tab_mn, st.tab_s, r, L, active);
      if (KERNEL == kSoftmaxBwd) W::softmax_bwd(u, p.data, p.codes, p.meta, r, L, active);
      u.sync();  // the next row may share a word / code byte with this one
    }
  }
};

// ---------------------------------------------------------------- 16-byte streaming
// Rows whose length is a multiple of the 16-byte vector.  A unit streams the row out of
// shared memory as many times as the arithmetic needs (shared memory has several times
// the bandwidth of an SM's share of HBM), so the GELU kernels keep nothing in registers
// and accept any row length; the softmax kernels keep NV vectors per lane.
constexpr uint32_t kMagicBits = 0x4B400000u;  // bit pattern of 1.5 * 2^23

template <int DT> struct V16;
template <> struct V16<kBF16> {
  static constexpr int EPA = 8;
  using Raw = uint4;
  struct MinMax {  // packed bfloat16x2 running min / max
    uint32_t mn, mx;
    __device__ __forceinline__ void init() { mn = 0x7F807F80u; mx = 0xFF80FF80u; }
    __device__ __forceinline__ void add(const Raw& r) {
      const uint32_t w[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        __nv_bfloat162 v = *(const __nv_bfloat162*)&w[k];
        __nv_bfloat162 a = __hmin2(*(__nv_bfloat162*)&mn, v), b = __hmax2(*(__nv_bfloat162*)&mx, v);
        mn = *(uint32_t*)&a;
        mx = *(uint32_t*)&b;
      }
    }
    __device__ __forceinline__ float lo() const {
      return fminf(__uint_as_float(mn << 16), __uint_as_float(mn & 0xffff0000u));
    }
    __device__ __forceinline__ float hi() const {
      return fmaxf(__uint_as_float(mx << 16), __uint_as_float(mx & 0xffff0000u));
    }
  };
  static __device__ __forceinline__ void widen(const Raw& r, float* v) {
    const uint32_t w[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      v[2 * k] = __uint_as_float(w[k] << 16);
      v[2 * k + 1] = __uint_as_float(w[k] & 0xffff0000u);
    }
  }
  // Rounds to bfloat16; leaves the values as written in v.
  static __device__ __forceinline__ Raw narrow(float* v) {
    uint32_t w[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      __nv_bfloat162 b = __floats2bfloat162_rn(v[2 * k], v[2 * k + 1]);
      w[k] = *(uint32_t*)&b;
      v[2 * k] = __uint_as_float(w[k] << 16);
      v[2 * k + 1] = __uint_as_float(w[k] & 0xffff0000u);
    }
    return make_uint4(w[0], w[1], w[2], w[3]);
  }
  static __device__ __forceinline__ uint32_t load_codes(const unsigned char* c, uint32_t j) {
    return *(const uint32_t*)(c + j * 4u);
  }
  static __device__ __forceinline__ void store_codes(unsigned char* c, uint32_t j, uint32_t bits) {
    *(uint32_t*)(c + j * 4u) = bits;
  }
};
template <> struct V16<kF32> {
  static constexpr int EPA = 4;
  using Raw = float4;
  struct MinMax {
    float mn, mx;
    __device__ __forceinline__ void init() { mn = INFINITY; mx = -INFINITY; }
    __device__ __forceinline__ void add(const Raw& r) {
      mn = fminf(fminf(mn, r.x), fminf(r.y, fminf(r.z, r.w)));
      mx = fmaxf(fmaxf(mx, r.x), fmaxf(r.y, fmaxf(r.z, r.w)));
    }
    __device__ __forceinline__ float lo() const { return mn; }
    __device__ __forceinline__ float hi() const { return mx; }
  };
  static __device__ __forceinline__ void widen(const Raw& r, float* v) {
    v[0] = r.x; v[1] = r.y; v[2] = r.z; v[3] = r.w;
  }
  static __device__ __forceinline__ Raw narrow(float* v) { return make_float4(v[0], v[1], v[2], v[3]); }
  static __device__ __forceinline__ uint32_t load_codes(const unsigned char* c, uint32_t j) {
    return *(const uint16_t*)(c + j * 2u);
  }
  static __device__ __forceinline__ void store_codes(unsigned char* c, uint32_t j, uint32_t bits) {
    *(uint16_t*)(c + j * 2u) = (uint16_t)bits;
  }
};

// Codes of N elements packed with one shift-add each: the rounded value sits in the low
// mantissa bits of (t + 1.5 * 2^23), whose other bits are a known constant.  Only the
// low 4N bits of `acc` are meaningful.
template <int N>
struct CodePacker {
  static constexpr uint32_t kOnes = N == 8 ? 0x11111111u : (N == 4 ? 0x1111u : 0x11u);
  uint32_t acc;
  __device__ __forceinline__ void init() { acc = 0u - kMagicBits * kOnes; }
  __device__ __forceinline__ void add(int k, float v, const QRange& q) {
    const float t = __fmul_rn(__fsub_rn(v, q.mn), q.inv);
    acc += __float_as_uint(__fadd_rn(t, 12582912.0f)) << (4 * k);
  }
};

// First pass of the activation forward over one row in shared memory: the row's exact minimum
// and its maximum "up to the clip" (exact when below `clip`, otherwise some value >= clip).
template <int DT, int UNIT_, int NVL>
__device__ __forceinline__ void act_row_extremes(Unit<UNIT_>& u, const unsigned char* row, uint32_t nv, float clip,
                                                 float& mn, float& mx) {
  using V = V16<DT>;
  if constexpr (DT == kBF16) {
    // The range of Eq. 8 is that of the CLIPPED row, so of the maximum only "at least the clip
    // value, or else its exact value" matters: it is taken over each lane's first vector, and
    // the whole row is searched only if that sample stays below the clip (a hidden vector of
    // thousands of activations practically never does).  The minimum is needed exactly -- it
    // also decides which form of the activation the second pass may use.  Packed bfloat16 pairs
    // throughout; (min, -max) are reduced together.
    auto min4 = [](uint32_t m, const uint4& v) {
      const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        const __nv_bfloat162 a = __hmin2(*(const __nv_bfloat162*)&m, *(const __nv_bfloat162*)&w[k]);
        m = *(const uint32_t*)&a;
      }
      return m;
    };
    auto max4 = [](uint32_t m, const uint4& v) {
      const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        const __nv_bfloat162 a = __hmax2(*(const __nv_bfloat162*)&m, *(const __nv_bfloat162*)&w[k]);
        m = *(const uint32_t*)&a;
      }
      return m;
    };
    auto lo = [](uint32_t w) { return __uint_as_float(w << 16); };
    auto hi = [](uint32_t w) { return __uint_as_float(w & 0xffff0000u); };
    uint32_t mn2 = 0x7F807F80u, mx2 = 0xFF80FF80u;
    if (NVL > 0) {
#pragma unroll
      for (int i = 0; i < NVL; ++i) {
        const uint4 v = *(const uint4*)(row + (u.ul + UNIT_ * i) * 16u);
        mn2 = min4(mn2, v);
        if (i == 0) mx2 = max4(mx2, v);
      }
    } else {
      if ((uint32_t)u.ul < nv) mx2 = max4(mx2, *(const uint4*)(row + u.ul * 16u));
#pragma unroll 4
      for (uint32_t j = u.ul; j < nv; j += UNIT_) mn2 = min4(mn2, *(const uint4*)(row + j * 16u));
    }
    const __nv_bfloat162 both = __floats2bfloat162_rn(fminf(lo(mn2), hi(mn2)), -fmaxf(lo(mx2), hi(mx2)));  // exact
    const uint32_t w = u.reduce_min_bf16x2(*(const uint32_t*)&both);
    mn = lo(w);
    mx = -hi(w);
    // The decision is the same in every lane of a unit; sub-warp units share their warp's
    // shuffles, so there the whole warp searches as soon as one of its units has to (a unit that
    // did not need it finds its exact maximum, which clips to the same value).
    bool search = mx < clip;
    if (UNIT_ < 32) search = __any_sync(0xffffffffu, search);
    if (search) {
      mx2 = 0xFF80FF80u;
      for (uint32_t j = u.ul; j < nv; j += UNIT_) mx2 = max4(mx2, *(const uint4*)(row + j * 16u));
      mx = u.template reduce<kOpMax>(fmaxf(lo(mx2), hi(mx2)));
    }
  } else {
    typename V::MinMax mm;
    mm.init();
    if (NVL > 0) {
#pragma unroll
      for (int i = 0; i < NVL; ++i) mm.add(*(const typename V::Raw*)(row + (u.ul + UNIT_ * i) * 16u));
    } else {
#pragma unroll 4
      for (uint32_t j = u.ul; j < nv; j += UNIT_) mm.add(*(const typename V::Raw*)(row + j * 16u));
    }
    mn = u.template reduce<kOpMin>(mm.lo());
    mx = u.template reduce<kOpMax>(mm.hi());
  }
}

// Eq. 8's range of a row clipped to +-clip, from the row's extremes: min / max of the clipped row
// = clipped min / max of the row (the clip is monotone).  A row that reaches both clip values has
// the same range as every other such row: its two quotients are constants, correctly rounded at
// compile time.
template <int ACT, int LEVELS>
__device__ __forceinline__ QRange clipped_qrange(float mn, float mx) {
  constexpr float kClip = Act<ACT>::kClipOf;
  const float cmn = fminf(fmaxf(mn, -kClip), kClip), cmx = fminf(fmaxf(mx, -kClip), kClip);
  QRange q;
  if (cmn == -kClip && cmx == kClip) {
    constexpr float kFullInv = (float)LEVELS / (2.0f * kClip), kFullS = (2.0f * kClip) / (float)LEVELS;
    q.mn = -kClip;
    q.inv = kFullInv;
    q.s = kFullS;
  } else {
    q = make_qrange(cmn, cmx, (float)LEVELS);
  }
  return q;
}

// NVL > 0 fixes the number of vectors per lane (row_len == NVL * UNIT * EPA), which lets
// the compiler drop every loop counter and bound check; NVL == 0 is the general loop.
template <int DT, int UNIT_, int NVL, int ACT>
struct StreamActFwd {
  static constexpr int kMaxRegs = 64;
  static constexpr int kKernel = ACT == kActGelu ? kGeluFwd : kSiluFwd;
  static constexpr float kActClip = Act<ACT>::kClipOf;
  static constexpr int UNIT = UNIT_;
  using V = V16<DT>;
  struct State {};
  static __device__ __forceinline__ void init(State&) {}
  static __device__ __forceinline__ uint32_t rows_per_group(uint32_t) { return 1u; }

  // FAST: the short bfloat16 form of the activation (two elements share one reciprocal), valid
  // on rows with no element below ActQuad::kQuadFloor (the caller knows the row minimum before
  // the second pass).
  template <bool FAST>
  static __device__ __forceinline__ void vec(unsigned char* row, unsigned char* crow, uint32_t j, const QRange& q) {
    // packed binary32 pairs throughout: one instruction per two elements
    const F2 min2 = f2_both(q.mn), inv2 = f2_both(q.inv), magic2 = f2_both(12582912.0f);
    uint32_t acc = 0u - kMagicBits * CodePacker<V::EPA>::kOnes;   // see CodePacker
    if constexpr (DT == kBF16) {
      const uint4 raw = *(const uint4*)(row + j * 16u);
      const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
      uint32_t o[4];
      F2 x[4];
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        x[k] = f2_from_bf16x2(w[k]);
        float t0, t1;
        f2_unpack(f2_add(f2_scaled(f2_clip(x[k], kActClip), min2, inv2), magic2), t0, t1);
        acc += __float_as_uint(t0) << (8 * k);
        acc += __float_as_uint(t1) << (8 * k + 4);
      }
      if constexpr (FAST) {
#pragma unroll
        for (int k = 0; k < 4; k += 2) {
          F2 ya, yb;
          ActQuad<ACT>::eval(x[k], x[k + 1], ya, yb);
          o[k] = f2_to_bf16x2(ya);
          o[k + 1] = f2_to_bf16x2(yb);
        }
      } else {
#pragma unroll
        for (int k = 0; k < 4; ++k) o[k] = f2_to_bf16x2(f2_act_general<ACT>(x[k]));
      }
      *(uint4*)(row + j * 16u) = make_uint4(o[0], o[1], o[2], o[3]);
    } else {
      const float4 raw = *(const float4*)(row + j * 16u);
      const float x[4] = {raw.x, raw.y, raw.z, raw.w};
      float y[4];
#pragma unroll
      for (int k = 0; k < 2; ++k) {
        float t0, t1;
        f2_unpack(f2_add(f2_scaled(f2_clip(f2_pack(x[2 * k], x[2 * k + 1]), kActClip), min2, inv2), magic2), t0, t1);
        acc += __float_as_uint(t0) << (8 * k);
        acc += __float_as_uint(t1) << (8 * k + 4);
        y[2 * k] = gelu_eval<DT, ACT>(x[2 * k]);
        y[2 * k + 1] = gelu_eval<DT, ACT>(x[2 * k + 1]);
      }
      *(float4*)(row + j * 16u) = make_float4(y[0], y[1], y[2], y[3]);
    }
    V::store_codes(crow, j, acc);
  }
  template <bool FAST>
  static __device__ __forceinline__ void second_pass(unsigned char* row, unsigned char* crow, int ul, uint32_t nv,
                                                     const QRange& q) {
    if (DT == kBF16 && !FAST) {
      // the rare rows with an element below the short form's range: kept rolled and small
#pragma unroll 1
      for (uint32_t j = ul; j < nv; j += UNIT_) vec<false>(row, crow, j, q);
    } else if (NVL > 0) {
#pragma unroll
      for (int i = 0; i < NVL; ++i) vec<FAST>(row, crow, ul + UNIT_ * i, q);
    } else {
#pragma unroll 2
      for (uint32_t j = ul; j < nv; j += UNIT_) vec<FAST>(row, crow, j, q);
    }
  }

  static __device__ __forceinline__ void group(Unit<UNIT_>& u, State&, const StagePtrs& p, float*, uint32_t r,
                                               bool active, uint32_t L) {
    if (UNIT_ >= 32 && !active) return;  // whole warps leave together
    const uint32_t nv = active ? L / V::EPA : 0u;
    unsigned char* row = p.data + (size_t)r * L * Io<DT>::kBytes;
    unsigned char* crow = p.codes + (size_t)r * (L / 2);
    float mn, mx;
    act_row_extremes<DT, UNIT_, NVL>(u, row, nv, kActClip, mn, mx);
    const QRange q = clipped_qrange<ACT, 15>(mn, mx);
    if (active && u.ul == 0) { p.meta[2 * r] = q.mn; p.meta[2 * r + 1] = q.s; }
    // mn is the same in every lane of the unit, so the branch does not diverge
    if (DT == kBF16 && mn >= ActQuad<ACT>::kQuadFloor) second_pass<true>(row, crow, u.ul, nv, q);
    else second_pass<false>(row, crow, u.ul, nv, q);
  }
};

template <int DT, int UNIT_, int NVL> using StreamGeluFwd = StreamActFwd<DT, UNIT_, NVL, kActGelu>;
template <int DT, int UNIT_, int NVL> using StreamSiluFwd = StreamActFwd<DT, UNIT_, NVL, kActSilu>;

// GELU backward.  With a whole warp on one row the 16 derivative values live one per
// lane (twice over) and are fetched with a shuffle indexed by the code; smaller units
// read them from a shared-memory table.
template <int DT, int UNIT_, int NVL, int ACT>
struct StreamActBwd {
  static constexpr int kMaxRegs = 64;
  static constexpr int kKernel = ACT == kActGelu ? kGeluBwd : kSiluBwd;
  static constexpr int UNIT = UNIT_;
  using V = V16<DT>;
  struct State {
    float tab_mn, tab_s, d;  // cached (min, s) and this lane's table entry
  };
  static __device__ __forceinline__ void init(State& st) {
    st.tab_mn = __int_as_float(0x7fc00000);
    st.tab_s = st.tab_mn;
    st.d = 0.0f;
  }
  static __device__ __forceinline__ uint32_t rows_per_group(uint32_t) { return 1u; }

  static __device__ __forceinline__ void group(Unit<UNIT_>& u, State& st, const StagePtrs& p, float* tab,
                                               uint32_t r, bool active, uint32_t L) {
    const float mn = active ? p.meta[2 * r] : st.tab_mn;
    const float s = active ? p.meta[2 * r + 1] : st.tab_s;
    // The 16 values of Eq. 12 this row can take, in binary64; kept while (min, s) repeat.
    if (mn != st.tab_mn || s != st.tab_s) {
      if (UNIT_ >= 32) {
        st.d = (float)act_derivative<ACT>((uint32_t)(u.ul & 15), mn, s);
      } else {
#pragma unroll
        for (int c = 0; c < 16; c += (UNIT_ < 16 ? UNIT_ : 16)) {
          const int code = c + u.ul;
          if (u.ul < 16 && code < 16) tab[code] = (float)act_derivative<ACT>((uint32_t)code, mn, s);
        }
      }
      st.tab_mn = mn;
      st.tab_s = s;
    }
    if (UNIT_ < 32) u.sync();
    if (UNIT_ >= 32 && !active) return;  // whole warps leave together
    const uint32_t nv = active ? L / V::EPA : 0u;
    unsigned char* row = p.data + (size_t)r * L * Io<DT>::kBytes;
    const unsigned char* crow = p.codes + (size_t)r * (L / 2);
    if (NVL > 0) {
#pragma unroll
      for (int i = 0; i < NVL; ++i) vec(st, tab, row, crow, u.ul + UNIT_ * i, true);
    } else {
      // every lane runs the same number of rounds so that the shuffles stay warp-wide
      const uint32_t rounds = (nv + UNIT_ - 1) / UNIT_;
#pragma unroll 2
      for (uint32_t it = 0; it < rounds; ++it) {
        const uint32_t j = it * UNIT_ + u.ul;
        vec(st, tab, row, crow, j, j < nv);
      }
    }
  }

  static __device__ __forceinline__ void vec(const State& st, const float* tab, unsigned char* row,
                                             const unsigned char* crow, uint32_t j, bool ok) {
    float v[V::EPA];
    uint32_t bits = 0;
    if (ok) {
      V::widen(*(const typename V::Raw*)(row + j * 16u), v);
      bits = V::load_codes(crow, j);
    }
#pragma unroll
    for (int k = 0; k < V::EPA; ++k) {
      float d;
      if (UNIT_ >= 32) d = __shfl_sync(0xffffffffu, st.d, (int)(bits >> (4 * k)));  // lane = code mod 16 (+16)
      else d = tab[(bits >> (4 * k)) & 0xFu];
      v[k] *= d;
    }
    if (ok) *(typename V::Raw*)(row + j * 16u) = V::narrow(v);
  }
};

template <int DT, int UNIT_, int NVL> using StreamGeluBwd = StreamActBwd<DT, UNIT_, NVL, kActGelu>;
template <int DT, int UNIT_, int NVL> using StreamSiluBwd = StreamActBwd<DT, UNIT_, NVL, kActSilu>;

// ---------------------------------------------------------------- Eq. 8 at 2 and 8 bits
// The streamed GELU kernels for code widths other than 4 (rows of whole 16-byte vectors,
// units of two or four warps).  A vector of EPA elements owns EPA * NBITS / 8 code bytes.
template <int N, int NBITS>
struct CodePackerBits {
  static constexpr int PER = 32 / NBITS;            // codes per 32-bit word
  static constexpr int W = (N + PER - 1) / PER;
  uint32_t acc[W];
  __device__ __forceinline__ void init() {
#pragma unroll
    for (int w = 0; w < W; ++w) {
      uint32_t ones = 0;
#pragma unroll
      for (int k = 0; k < PER; ++k)
        if (w * PER + k < N) ones |= 1u << (NBITS * k);
      acc[w] = 0u - kMagicBits * ones;
    }
  }
  __device__ __forceinline__ void add(int k, float v, const QRange& q) {
    const float t = __fmul_rn(__fsub_rn(v, q.mn), q.inv);
    acc[k / PER] += __float_as_uint(__fadd_rn(t, 12582912.0f)) << (NBITS * (k % PER));
  }
};

template <int DT, int NBITS>
struct CodeIo {
  static constexpr int EPA = V16<DT>::EPA;
  static constexpr int BYTES = EPA * NBITS / 8;     // 1, 2, 4 or 8 code bytes per vector
  static constexpr int W = (BYTES + 3) / 4;
  static __device__ __forceinline__ void store(unsigned char* c, uint32_t j, const uint32_t* w) {
    if (BYTES == 1) c[j] = (unsigned char)w[0];
    if (BYTES == 2) *(uint16_t*)(c + j * 2u) = (uint16_t)w[0];
    if (BYTES == 4) *(uint32_t*)(c + j * 4u) = w[0];
    if (BYTES == 8) *(uint2*)(c + j * 8u) = make_uint2(w[0], w[W - 1]);
  }
  static __device__ __forceinline__ void load(const unsigned char* c, uint32_t j, uint32_t* w) {
    if (BYTES == 1) w[0] = c[j];
    if (BYTES == 2) w[0] = *(const uint16_t*)(c + j * 2u);
    if (BYTES == 4) w[0] = *(const uint32_t*)(c + j * 4u);
    if (BYTES == 8) {
      const uint2 t = *(const uint2*)(c + j * 8u);
      w[0] = t.x;
      w[W - 1] = t.y;
    }
  }
};

template <int DT, int UNIT_, int ACT, int NBITS>
struct StreamActFwdBits {
  static_assert(UNIT_ >= 64 && (NBITS == 2 || NBITS == 8), "multi-warp units, 2 or 8 bits");
  static constexpr int kMaxRegs = 64;
  static constexpr int kKernel = ACT == kActGelu ? kGeluFwd : kSiluFwd;
  static constexpr float kActClip = Act<ACT>::kClipOf;
  static constexpr int UNIT = UNIT_;
  using V = V16<DT>;
  using C = CodeIo<DT, NBITS>;
  struct State {};
  static __device__ __forceinline__ void init(State&) {}
  static __device__ __forceinline__ uint32_t rows_per_group(uint32_t) { return 1u; }

  static __device__ __forceinline__ void group(Unit<UNIT_>& u, State&, const StagePtrs& p, float*, uint32_t r,
                                               bool active, uint32_t L) {
    if (!active) return;  // whole warps leave together
    const uint32_t nv = L / V::EPA;
    unsigned char* row = p.data + (size_t)r * L * Io<DT>::kBytes;
    unsigned char* crow = p.codes + (size_t)r * (L / V::EPA) * C::BYTES;
    float mn, mx;
    act_row_extremes<DT, UNIT_, 0>(u, row, nv, kActClip, mn, mx);
    const QRange q = clipped_qrange<ACT, (1 << NBITS) - 1>(mn, mx);
    if (u.ul == 0) { p.meta[2 * r] = q.mn; p.meta[2 * r + 1] = q.s; }
#pragma unroll 2
    for (uint32_t j = u.ul; j < nv; j += UNIT_) {
      float v[V::EPA];
      V::widen(*(const typename V::Raw*)(row + j * 16u), v);
      CodePackerBits<V::EPA, NBITS> pk;
      pk.init();
#pragma unroll
      for (int k = 0; k < V::EPA; ++k) {
        pk.add(k, fminf(fmaxf(v[k], -kActClip), kActClip), q);
        v[k] = gelu_eval<DT, ACT>(v[k]);
      }
      *(typename V::Raw*)(row + j * 16u) = V::narrow(v);
      C::store(crow, j, pk.acc);
    }
  }
};

// Backward: the 2^NBITS derivative values of a row.  Four values sit one per lane (eight
// times over) and are fetched with a shuffle; 256 values go to a table of the unit's own
// in shared memory.  Either is kept while (min, s) repeat from row to row.
template <int DT, int UNIT_, int ACT, int NBITS>
struct StreamActBwdBits {
  static_assert(UNIT_ >= 64 && (NBITS == 2 || NBITS == 8), "multi-warp units, 2 or 8 bits");
  static constexpr int kMaxRegs = 64;
  static constexpr int kKernel = ACT == kActGelu ? kGeluBwd : kSiluBwd;
  static constexpr int UNIT = UNIT_;
  static constexpr int kTabFloats = NBITS == 8 ? 256 : 16;
  using V = V16<DT>;
  using C = CodeIo<DT, NBITS>;
  struct State {
    float tab_mn, tab_s, d;
  };
  static __device__ __forceinline__ void init(State& st) {
    st.tab_mn = __int_as_float(0x7fc00000);  // NaN: nothing cached yet
    st.tab_s = st.tab_mn;
    st.d = 0.0f;
  }
  static __device__ __forceinline__ uint32_t rows_per_group(uint32_t) { return 1u; }

  static __device__ __forceinline__ void group(Unit<UNIT_>& u, State& st, const StagePtrs& p, float* tab,
                                               uint32_t r, bool active, uint32_t L) {
    if (!active) return;  // whole warps leave together
    const float mn = p.meta[2 * r];
    const float s = p.meta[2 * r + 1];
    if (mn != st.tab_mn || s != st.tab_s) {  // the same decision in every lane of the unit
      if (NBITS == 2) {
        st.d = (float)act_derivative<ACT>((uint32_t)(u.ul & 3), mn, s);
      } else {
        u.sync();  // the previous row's reads of the table are over
        for (int c = u.ul; c < 256; c += UNIT_) tab[c] = (float)act_derivative<ACT>((uint32_t)c, mn, s);
        u.sync();
      }
      st.tab_mn = mn;
      st.tab_s = s;
    }
    const uint32_t nv = L / V::EPA;
    unsigned char* row = p.data + (size_t)r * L * Io<DT>::kBytes;
    const unsigned char* crow = p.codes + (size_t)r * (L / V::EPA) * C::BYTES;
    // every lane runs the same number of rounds so that the shuffles stay warp-wide
    const uint32_t rounds = (nv + UNIT_ - 1) / UNIT_;
#pragma unroll 2
    for (uint32_t it = 0; it < rounds; ++it) {
      const uint32_t j = it * UNIT_ + u.ul;
      const bool ok = j < nv;
      float v[V::EPA];
      uint32_t w[C::W] = {};
      if (ok) {
        V::widen(*(const typename V::Raw*)(row + j * 16u), v);
        C::load(crow, j, w);
      }
#pragma unroll
      for (int k = 0; k < V::EPA; ++k) {
        constexpr int PER = 32 / NBITS;
        const uint32_t code = w[k / PER] >> (NBITS * (k % PER));
        float d;
        if (NBITS == 2) d = __shfl_sync(0xffffffffu, st.d, (int)code);  // lane = code mod 4 (+4, +8, ...)
        else d = tab[code & 0xFFu];
        v[k] *= d;
      }
      if (ok) *(typename V::Raw*)(row + j * 16u) = V::narrow(v);
    }
  }
};

// Floats of derivative table a policy wants per unit (16 unless it says otherwise).
template <class W, class = void> struct TabFloats { static constexpr int value = 16; };
template <class W> struct TabFloats<W, std::void_t<decltype(W::kTabFloats)>> { static constexpr int value = W::kTabFloats; };

// Register cap of the streamed softmax kernels by elements held per lane (the planner
// derives the CTAs that fit an SM from the same number).
constexpr int softmax_stream_regs(int dt, int held) {
  return held >= 64 ? 128 : (held >= 32 ? (dt == kBF16 ? 112 : 128) : 80);
}

// Softmax forward on 16-byte vectors, NV vectors per lane kept in registers.  Short rows
// leave a lane with little work between the four row reductions, so a unit takes RPU rows
// at a time and walks them phase by phase: each row's shuffle latency hides behind the
// other rows' arithmetic.
template <int DT, int UNIT_, int NV>
struct StreamSoftmaxFwd {
  static constexpr int kMaxRegs = softmax_stream_regs(DT, NV * V16<DT>::EPA);
  static constexpr int kKernel = kSoftmaxFwd;
  static constexpr int UNIT = UNIT_;
  using V = V16<DT>;
  static constexpr int EPA = V::EPA;
  static constexpr int RPU = NV * EPA <= 8 ? 4 : (NV * EPA <= 16 ? 2 : 1);  // rows per unit per round
  struct State {};
  static __device__ __forceinline__ void init(State&) {}
  static __device__ __forceinline__ uint32_t rows_per_group(uint32_t) { return RPU; }

  // All binary32 arithmetic runs on packed pairs (one instruction per two elements).
  static constexpr int NP = EPA / 2;  // pairs per vector
  static __device__ __forceinline__ uint32_t hmax2u(uint32_t a, uint32_t b) {
    __nv_bfloat162 r = __hmax2(*(__nv_bfloat162*)&a, *(__nv_bfloat162*)&b);
    return *(uint32_t*)&r;
  }
  static __device__ __forceinline__ uint32_t hmin2u(uint32_t a, uint32_t b) {
    __nv_bfloat162 r = __hmin2(*(__nv_bfloat162*)&a, *(__nv_bfloat162*)&b);
    return *(uint32_t*)&r;
  }

  static __device__ __forceinline__ void group(Unit<UNIT_>& u, State&, const StagePtrs& p, float*, uint32_t grp,
                                               bool active, uint32_t L) {
    const uint32_t nv = active ? L / EPA : 0u;
    const uint32_t r0 = grp * RPU;
    F2 e[RPU][NV][NP];
    float m[RPU], z[RPU], mn[RPU], mx[RPU];
    const F2 ninf2 = f2_both(-INFINITY);
#pragma unroll
    for (int rr = 0; rr < RPU; ++rr) {
      const unsigned char* row = p.data + (size_t)(r0 + rr) * L * Io<DT>::kBytes;
      m[rr] = -INFINITY;
      uint32_t m2 = 0xFF80FF80u;  // bfloat16: packed running maximum
#pragma unroll
      for (int i = 0; i < NV; ++i) {
        const uint32_t j = u.ul + UNIT_ * i;
        if (j < nv) {
          if constexpr (DT == kBF16) {
            const uint4 raw = *(const uint4*)(row + j * 16u);
            const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
            for (int k = 0; k < 4; ++k) {
              m2 = hmax2u(m2, w[k]);
              e[rr][i][k] = f2_from_bf16x2(w[k]);
            }
          } else {
            const float4 raw = *(const float4*)(row + j * 16u);
            m[rr] = fmaxf(fmaxf(m[rr], raw.x), fmaxf(raw.y, fmaxf(raw.z, raw.w)));
            e[rr][i][0] = f2_pack(raw.x, raw.y);
            e[rr][i][1] = f2_pack(raw.z, raw.w);
          }
        } else {
#pragma unroll
          for (int k = 0; k < NP; ++k) e[rr][i][k] = ninf2;
        }
      }
      if constexpr (DT == kBF16) m[rr] = fmaxf(__uint_as_float(m2 << 16), __uint_as_float(m2 & 0xffff0000u));
    }
    constexpr bool kPackRows = DT == kBF16 && RPU >= 2 && UNIT_ <= 32;  // two rows share a shuffle chain
    if constexpr (DT == kBF16 && kPackRows) {
      // the maxima of two rows are bfloat16 values: one shuffle chain for the packed pair
#pragma unroll
      for (int rr = 0; rr < RPU; rr += 2) {
        __nv_bfloat162 pm = __floats2bfloat162_rn(m[rr], m[rr + 1]);
        uint32_t w = *(uint32_t*)&pm;
#pragma unroll
        for (int o = UNIT_ / 2; o > 0; o >>= 1) w = hmax2u(w, __shfl_xor_sync(0xffffffffu, w, o));
        m[rr] = __uint_as_float(w << 16);
        m[rr + 1] = __uint_as_float(w & 0xffff0000u);
      }
    } else {
#pragma unroll
      for (int rr = 0; rr < RPU; ++rr) m[rr] = u.template reduce<kOpMax>(m[rr]);
    }
#pragma unroll
    for (int rr = 0; rr < RPU; ++rr)
      if (!active) m[rr] = 0.0f;
    constexpr float kLog2e = 1.4426950408889634f;
    const F2 k2 = f2_both(kLog2e);
#pragma unroll
    for (int rr = 0; rr < RPU; ++rr) {
      // bfloat16: the exponent's argument is one fused multiply-add (the result is rounded to 8
      // bits); binary32: the difference, then the product (see exp_eval)
      const F2 c2 = f2_both(DT == kBF16 ? -m[rr] * kLog2e : m[rr]);
      F2 z2 = f2_both(0.0f);
#pragma unroll
      for (int i = 0; i < NV; ++i)
#pragma unroll
        for (int k = 0; k < NP; ++k) {
          float a0, a1;
          f2_unpack(DT == kBF16 ? f2_fma(e[rr][i][k], k2, c2) : f2_mul(k2, f2_sub(e[rr][i][k], c2)), a0, a1);
          e[rr][i][k] = f2_pack(ex2_approx(a0), ex2_approx(a1));
          z2 = f2_add(z2, e[rr][i][k]);
        }
      float z0, z1;
      f2_unpack(z2, z0, z1);
      z[rr] = z0 + z1;
    }
    if constexpr (kPackRows) {
      // the sums of two rows go down the shuffles together: one packed addition per step
#pragma unroll
      for (int rr = 0; rr < RPU; rr += 2) {
        F2 z2 = f2_pack(z[rr], z[rr + 1]);
#pragma unroll
        for (int o = UNIT_ / 2; o > 0; o >>= 1) {
          float x0, x1;
          f2_unpack(z2, x0, x1);
          z2 = f2_add(z2, f2_pack(__shfl_xor_sync(0xffffffffu, x0, o), __shfl_xor_sync(0xffffffffu, x1, o)));
        }
        f2_unpack(z2, z[rr], z[rr + 1]);
      }
    } else {
#pragma unroll
      for (int rr = 0; rr < RPU; ++rr) z[rr] = u.template reduce<kOpSum>(z[rr]);
    }
#pragma unroll
    for (int rr = 0; rr < RPU; ++rr) {
      unsigned char* row = p.data + (size_t)(r0 + rr) * L * Io<DT>::kBytes;
      const float zz = active ? z[rr] : 1.0f;
      float rz;
      if constexpr (DT == kBF16) {
        const float ra = rcp_approx(zz);  // about an ulp after the correction step; y keeps 8 bits
        rz = __fmaf_rn(__fmaf_rn(-zz, ra, 1.0f), ra, ra);
      } else {
        rz = __fdiv_rn(1.0f, zz);
      }
      const F2 rz2 = f2_both(rz);
      uint32_t mn2 = 0x7F807F80u, mx2 = 0xFF80FF80u;
      mn[rr] = INFINITY;
      mx[rr] = -INFINITY;
#pragma unroll
      for (int i = 0; i < NV; ++i) {
        const uint32_t j = u.ul + UNIT_ * i;
        if (j < nv) {
          if constexpr (DT == kBF16) {
            uint32_t w[4];
#pragma unroll
            for (int k = 0; k < 4; ++k) {
              w[k] = f2_to_bf16x2(f2_mul(e[rr][i][k], rz2));
              e[rr][i][k] = f2_from_bf16x2(w[k]);  // y as written
              mn2 = hmin2u(mn2, w[k]);
              mx2 = hmax2u(mx2, w[k]);
            }
            *(uint4*)(row + j * 16u) = make_uint4(w[0], w[1], w[2], w[3]);
          } else {
            float y[4];
#pragma unroll
            for (int k = 0; k < 2; ++k) {
              e[rr][i][k] = f2_mul(e[rr][i][k], rz2);
              f2_unpack(e[rr][i][k], y[2 * k], y[2 * k + 1]);
            }
            *(float4*)(row + j * 16u) = make_float4(y[0], y[1], y[2], y[3]);
            mn[rr] = fminf(fminf(mn[rr], y[0]), fminf(y[1], fminf(y[2], y[3])));
            mx[rr] = fmaxf(fmaxf(mx[rr], y[0]), fmaxf(y[1], fmaxf(y[2], y[3])));
          }
        }
      }
      if constexpr (DT == kBF16) {
        mn[rr] = fminf(__uint_as_float(mn2 << 16), __uint_as_float(mn2 & 0xffff0000u));
        mx[rr] = fmaxf(__uint_as_float(mx2 << 16), __uint_as_float(mx2 & 0xffff0000u));
      }
    }
#pragma unroll
    for (int rr = 0; rr < RPU; ++rr) {
      if constexpr (DT == kBF16 && UNIT_ <= 32) {
        reduce_minmax_bf16<UNIT_>(mn[rr], mx[rr]);
      } else {
        mn[rr] = u.template reduce<kOpMin>(mn[rr]);
        mx[rr] = u.template reduce<kOpMax>(mx[rr]);
      }
    }
    const F2 magic2 = f2_both(12582912.0f);
    // Eq. 8's two correctly rounded quotients per row (15 / d and d / 15).  A unit that walks
    // several rows forms them for all of its rows together: lane l takes quotient l (row l / 2;
    // even l: 15 / d, odd l: d / 15), in as many divisions as it takes the unit's lanes to cover
    // 2 * RPU quotients, and shuffles hand them round.
    constexpr int NDIV = kPackRows ? (2 * RPU + UNIT_ - 1) / UNIT_ : 1;
    float quo[NDIV];
    if constexpr (kPackRows) {
#pragma unroll
      for (int dv = 0; dv < NDIV; ++dv) {
        const int slot = dv * UNIT_ + u.ul;
        float d = 1.0f;
#pragma unroll
        for (int rr = 0; rr < RPU; ++rr)
          if ((slot >> 1) == rr) d = __fsub_rn(mx[rr], mn[rr]);
        const bool odd = (slot & 1) != 0;
        quo[dv] = __fdiv_rn(odd ? d : kLevels, odd ? kLevels : d);
        if (d == 0.0f) quo[dv] = 0.0f;  // a constant row: inv = s = 0
      }
    }
    const int base = threadIdx.x & 31 & ~((UNIT_ < 32 ? UNIT_ : 32) - 1);
#pragma unroll
    for (int rr = 0; rr < RPU; ++rr) {
      const uint32_t r = r0 + rr;
      unsigned char* crow = p.codes + (size_t)r * (L / 2);
      QRange q;
      if constexpr (kPackRows) {
        q.mn = mn[rr];
        q.inv = __shfl_sync(0xffffffffu, quo[(2 * rr) / UNIT_], base + (2 * rr) % UNIT_);
        q.s = __shfl_sync(0xffffffffu, quo[(2 * rr + 1) / UNIT_], base + (2 * rr + 1) % UNIT_);
      } else {
        q = make_qrange(mn[rr], mx[rr]);
      }
      if (active && u.ul == 0) { p.meta[2 * r] = q.mn; p.meta[2 * r + 1] = q.s; }
      const F2 min2 = f2_both(q.mn), inv2 = f2_both(q.inv);
#pragma unroll
      for (int i = 0; i < NV; ++i) {
        const uint32_t j = u.ul + UNIT_ * i;
        if (j < nv) {
          uint32_t acc = 0u - kMagicBits * CodePacker<EPA>::kOnes;  // see CodePacker
#pragma unroll
          for (int k = 0; k < NP; ++k) {
            float t0, t1;
            f2_unpack(f2_add(f2_scaled(e[rr][i][k], min2, inv2), magic2), t0, t1);
            acc += __float_as_uint(t0) << (8 * k);
            acc += __float_as_uint(t1) << (8 * k + 4);
          }
          V::store_codes(crow, j, acc);
        }
      }
    }
  }
};

template <int DT, int UNIT_, int NV>
struct StreamSoftmaxBwd {
  static constexpr int kMaxRegs = softmax_stream_regs(DT, NV * V16<DT>::EPA);
  static constexpr int kKernel = kSoftmaxBwd;
  static constexpr int UNIT = UNIT_;
  using V = V16<DT>;
  static constexpr int EPA = V::EPA;
  struct State {};
  static __device__ __forceinline__ void init(State&) {}
  static __device__ __forceinline__ uint32_t rows_per_group(uint32_t) { return 1u; }

  static __device__ __forceinline__ void group(Unit<UNIT_>& u, State&, const StagePtrs& p, float*, uint32_t r,
                                               bool active, uint32_t L) {
    const uint32_t nv = active ? L / EPA : 0u;
    unsigned char* row = p.data + (size_t)r * L * Io<DT>::kBytes;
    const unsigned char* crow = p.codes + (size_t)r * (L / 2);
    const float mn = active ? p.meta[2 * r] : 0.0f;
    const float s = active ? p.meta[2 * r + 1] : 0.0f;
    float g[NV][EPA], yh[NV][EPA];
    float dot = 0.0f;
#pragma unroll
    for (int i = 0; i < NV; ++i) {
      const uint32_t j = u.ul + UNIT_ * i;
      if (j < nv) {
        V::widen(*(const typename V::Raw*)(row + j * 16u), g[i]);
        const uint32_t bits = V::load_codes(crow, j);
#pragma unroll
        for (int k = 0; k < EPA; ++k) {
          yh[i][k] = dequant((bits >> (4 * k)) & 0xFu, mn, s);
          dot = fmaf(g[i][k], yh[i][k], dot);
        }
      }
    }
    dot = u.template reduce<kOpSum>(dot);
#pragma unroll
    for (int i = 0; i < NV; ++i) {
      const uint32_t j = u.ul + UNIT_ * i;
      if (j < nv) {
        float v[EPA];
#pragma unroll
        for (int k = 0; k < EPA; ++k) v[k] = yh[i][k] * (g[i][k] - dot);
        *(typename V::Raw*)(row + j * 16u) = V::narrow(v);
      }
    }
  }
};

// ---------------------------------------------------------------- softmax rows of any length
// Rows that are not a whole number of 16-byte vectors (attention widths such as 49, 145,
// 198, 577, 1025) or too long to hold in registers.  The tile is still read in ALIGNED
// 16-byte vectors: a row's first and last vector may hold elements of its neighbours, which
// are masked out of the arithmetic and never written (interior vectors leave with one
// 16-byte store, boundary vectors element by element, so two units never write the same
// bytes).  Nothing is held in registers: the row is streamed from shared memory once per
// phase, and the exponentials are evaluated twice (sum, then output) rather than kept in a
// narrower type.  With an odd row length two consecutive rows share a code byte: each merges
// its own nibble into it atomically, so rows need no particular order.
template <int DT>
struct AnyRow {
  using V = V16<DT>;
  static constexpr int EPA = V::EPA;
  static constexpr uint32_t kFull = (1u << EPA) - 1u;
  uint32_t v0, v1;    // first and last vector (tile-relative) that hold elements of the row
  uint32_t head;      // elements of v0 before the row
  uint32_t tail;      // elements of v1 inside the row (1..EPA)
  __device__ __forceinline__ void set(uint32_t r, uint32_t L) {
    const uint32_t e0 = r * L;
    v0 = e0 / EPA;
    v1 = (e0 + L - 1) / EPA;
    head = e0 - v0 * EPA;
    tail = e0 + L - v1 * EPA;
  }
  __device__ __forceinline__ uint32_t mask(uint32_t j) const {
    uint32_t m = kFull;
    if (j == v0) m &= kFull << head;
    if (j == v1) m &= (1u << tail) - 1u;
    return m;
  }
  // Writes the elements of vector j named by msk (raw: the vector's 16 bytes).
  static __device__ __forceinline__ void store(unsigned char* data, uint32_t j, const typename V::Raw& raw, uint32_t msk) {
    if (msk == kFull) {
      *(typename V::Raw*)(data + j * 16u) = raw;
      return;
    }
    const uint32_t* w = (const uint32_t*)&raw;
#pragma unroll
    for (int k = 0; k < EPA; ++k) {
      if (msk >> k & 1u) {
        if (DT == kBF16) *(uint16_t*)(data + j * 16u + 2 * k) = (uint16_t)(w[k >> 1] >> (16 * (k & 1)));
        else *(uint32_t*)(data + j * 16u + 4 * k) = w[k];
      }
    }
  }
};

// Calls f(j, mask, is_interior) for the vectors of a row that this lane owns.  The "edge"
// vectors are those that share a 32-bit word of CODES with the row's first or last vector
// (VPW vectors share a word; 1 if a vector's codes fill whole words): only there can
// another row's unit write the same word, so the forward kernels write codes atomically
// there and with plain stores everywhere else -- no word ever sees both kinds of access.
// The interior vectors go round the unit's lanes with no mask at all; the edge vectors are
// dealt out to the lanes in ONE divergent section, so that the masked code runs once per
// phase.  Every phase of a kernel must use the same VPW (a lane reads back what it wrote).
template <int DT, int UNIT_, int VPW = 1, class F>
__device__ __forceinline__ void any_row_vectors(const AnyRow<DT>& g, int ul, bool active, F&& f) {
  if (!active) return;
  const uint32_t lo_last = min(g.v1, (g.v0 / VPW + 1u) * VPW - 1u);   // last vector of the low edge group
  const uint32_t hi_first = max(lo_last + 1u, (g.v1 / VPW) * VPW);     // first vector of the high edge group
  for (uint32_t j = lo_last + 1u + (uint32_t)ul; j < hi_first; j += UNIT_) f(j, AnyRow<DT>::kFull, std::true_type{});
  const uint32_t n_lo = lo_last - g.v0 + 1u, n_hi = g.v1 >= hi_first ? g.v1 - hi_first + 1u : 0u;
  for (uint32_t t = (uint32_t)ul; t < n_lo + n_hi; t += UNIT_) {
    const uint32_t j = t < n_lo ? g.v0 + t : hi_first + (t - n_lo);
    f(j, g.mask(j), std::false_type{});
  }
}

// Merges the codes of the elements of vector j named by msk into the code bytes, with
// atomics on the enclosing 32-bit words (acc: the vector's packed codes, NBITS each).
template <int NBITS, int EPA>
__device__ __forceinline__ void any_merge_codes(unsigned char* codes, uint32_t j, const uint32_t* acc, uint32_t msk) {
  constexpr int PER = 32 / NBITS;                 // codes per word of acc
  constexpr int BYTES = EPA * NBITS / 8;          // code bytes of one vector
  constexpr int W = (BYTES + 3) / 4;
  constexpr uint32_t kCodeMask = (1u << NBITS) - 1u;
  uint32_t own[W] = {};
#pragma unroll
  for (int k = 0; k < EPA; ++k)
    if (msk >> k & 1u) own[k / PER] |= kCodeMask << (NBITS * (k % PER));
  if (BYTES >= 4) {
#pragma unroll
    for (int w = 0; w < W; ++w) {
      unsigned int* word = (unsigned int*)codes + j * W + w;
      if (own[w] != 0u) {
        atomicAnd(word, ~own[w]);
        atomicOr(word, acc[w] & own[w]);
      }
    }
  } else {
    const uint32_t off = j * BYTES;
    unsigned int* word = (unsigned int*)(codes + (off & ~3u));
    const uint32_t sh = 8u * (off & 3u);
    atomicAnd(word, ~(own[0] << sh));
    atomicOr(word, (acc[0] & own[0]) << sh);
  }
}

template <int DT, int UNIT_>
struct AnySoftmaxFwd {
  static constexpr int kMaxRegs = 80;  // 2 CTAs of 8 + 1 warps per SM
  static constexpr int kKernel = kSoftmaxFwd;
  static constexpr int UNIT = UNIT_;
  using V = V16<DT>;
  using R = AnyRow<DT>;
  static constexpr int EPA = V::EPA;
  static constexpr int NP = EPA / 2;              // packed binary32 pairs per vector
  static constexpr int kVPW = EPA == 8 ? 1 : 2;  // vectors per 32-bit word of codes
  struct State {};
  static __device__ __forceinline__ void init(State&) {}
  static __device__ __forceinline__ uint32_t rows_per_group(uint32_t) { return 1u; }

  // The vector's elements as packed binary32 pairs (exact).
  static __device__ __forceinline__ void pairs_of(const typename V::Raw& raw, F2* x) {
    if constexpr (DT == kBF16) {
      const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
      for (int k = 0; k < 4; ++k) x[k] = f2_from_bf16x2(w[k]);
    } else {
      x[0] = f2_pack(raw.x, raw.y);
      x[1] = f2_pack(raw.z, raw.w);
    }
  }
  // e^(x - m) for the vector's elements: bfloat16 with one fused multiply-add per exponent
  // argument (c2 = -m log2 e), binary32 with the difference, then the product (c2 = m).
  static __device__ __forceinline__ void exps_of(const typename V::Raw& raw, F2 c2, F2* e) {
    const F2 k2 = f2_both(1.4426950408889634f);
    pairs_of(raw, e);
#pragma unroll
    for (int k = 0; k < NP; ++k) {
      float a, b;
      f2_unpack(DT == kBF16 ? f2_fma(e[k], k2, c2) : f2_mul(k2, f2_sub(e[k], c2)), a, b);
      e[k] = f2_pack(ex2_approx(a), ex2_approx(b));
    }
  }
  // Keeps the elements named by msk (bit 2k: low half of pair k, bit 2k + 1: high half), others become `other`.
  static __device__ __forceinline__ F2 masked(F2 v, uint32_t msk, int k, float other) {
    float a, b;
    f2_unpack(v, a, b);
    return f2_pack((msk >> (2 * k) & 1u) ? a : other, (msk >> (2 * k + 1) & 1u) ? b : other);
  }

  static __device__ __forceinline__ void row(Unit<UNIT_>& u, const StagePtrs& p, uint32_t r, bool active, uint32_t L) {
    R g;
    g.set(r, L);
    const int ul = u.ul;
    // ---- row maximum (interior vectors of bfloat16 rows: packed maxima on the raw words)
    float m = -INFINITY;
    typename V::MinMax pm;
    pm.init();
    any_row_vectors<DT, UNIT_, kVPW>(g, ul, active, [&](uint32_t j, uint32_t msk, auto interior) {
      const typename V::Raw raw = *(const typename V::Raw*)(p.data + j * 16u);
      if constexpr (decltype(interior)::value) {
        pm.add(raw);
      } else {
        float v[EPA];
        V::widen(raw, v);
#pragma unroll
        for (int k = 0; k < EPA; ++k) m = fmaxf(m, (msk >> k & 1u) ? v[k] : -INFINITY);
      }
    });
    m = u.template reduce<kOpMax>(fmaxf(m, pm.hi()));
    if (!active) m = 0.0f;
    const F2 c2 = f2_both(DT == kBF16 ? -m * 1.4426950408889634f : m);
    // ---- sum of exponentials
    F2 z2 = f2_both(0.0f);
    any_row_vectors<DT, UNIT_, kVPW>(g, ul, active, [&](uint32_t j, uint32_t msk, auto interior) {
      F2 e[NP];
      exps_of(*(const typename V::Raw*)(p.data + j * 16u), c2, e);
#pragma unroll
      for (int k = 0; k < NP; ++k) {
        if constexpr (decltype(interior)::value) z2 = f2_add(z2, e[k]);
        else z2 = f2_add(z2, masked(e[k], msk, k, 0.0f));
      }
    });
    float z0, z1;
    f2_unpack(z2, z0, z1);
    const float z = u.template reduce<kOpSum>(z0 + z1);
    const F2 rz2 = f2_both(__fdiv_rn(1.0f, active ? z : 1.0f));
    // ---- y, written in place, and the range of y as written
    float mn = INFINITY, mx = -INFINITY;
    typename V::MinMax py;
    py.init();
    any_row_vectors<DT, UNIT_, kVPW>(g, ul, active, [&](uint32_t j, uint32_t msk, auto interior) {
      F2 e[NP];
      exps_of(*(const typename V::Raw*)(p.data + j * 16u), c2, e);
      typename V::Raw yw;
      if constexpr (DT == kBF16) {
        yw = make_uint4(f2_to_bf16x2(f2_mul(e[0], rz2)), f2_to_bf16x2(f2_mul(e[1], rz2)), f2_to_bf16x2(f2_mul(e[2], rz2)),
                        f2_to_bf16x2(f2_mul(e[3], rz2)));
      } else {
        float a, b, c, d;
        f2_unpack(f2_mul(e[0], rz2), a, b);
        f2_unpack(f2_mul(e[1], rz2), c, d);
        yw = make_float4(a, b, c, d);
      }
      if constexpr (decltype(interior)::value) {
        *(typename V::Raw*)(p.data + j * 16u) = yw;
        py.add(yw);
      } else {
        R::store(p.data, j, yw, msk);
        float v[EPA];
        V::widen(yw, v);  // y as written
#pragma unroll
        for (int k = 0; k < EPA; ++k) {
          mn = fminf(mn, (msk >> k & 1u) ? v[k] : INFINITY);
          mx = fmaxf(mx, (msk >> k & 1u) ? v[k] : -INFINITY);
        }
      }
    });
    mn = u.template reduce<kOpMin>(fminf(mn, py.lo()));
    mx = u.template reduce<kOpMax>(fmaxf(mx, py.hi()));
    const QRange q = make_qrange(mn, mx);
    if (active && ul == 0) { p.meta[2 * r] = q.mn; p.meta[2 * r + 1] = q.s; }
    const F2 min2 = f2_both(q.mn), inv2 = f2_both(q.inv), magic2 = f2_both(12582912.0f);
    // ---- codes of y as written (each lane reads back the vectors it wrote itself)
    any_row_vectors<DT, UNIT_, kVPW>(g, ul, active, [&](uint32_t j, uint32_t msk, auto interior) {
      F2 y[NP];
      pairs_of(*(const typename V::Raw*)(p.data + j * 16u), y);
      uint32_t acc = 0u - kMagicBits * CodePacker<EPA>::kOnes;  // see CodePacker
#pragma unroll
      for (int k = 0; k < NP; ++k) {
        // a neighbour's element codes as 0 (it is replaced by the minimum)
        const F2 v = decltype(interior)::value ? y[k] : masked(y[k], msk, k, q.mn);
        float t0, t1;
        f2_unpack(f2_add(f2_scaled(v, min2, inv2), magic2), t0, t1);
        acc += __float_as_uint(t0) << (8 * k);
        acc += __float_as_uint(t1) << (8 * k + 4);
      }
      if constexpr (decltype(interior)::value) V::store_codes(p.codes, j, acc);
      else any_merge_codes<4, EPA>(p.codes, j, &acc, msk);
    });
  }

  static __device__ __forceinline__ void group(Unit<UNIT_>& u, State&, const StagePtrs& p, float*, uint32_t grp,
                                               bool active, uint32_t L) {
    if (UNIT_ >= 32 && !active) return;  // whole warps (and whole multi-warp units) leave together
    row(u, p, active ? grp : 0u, active, L);
    if (UNIT_ < 32) u.sync();
  }
};

template <int DT, int UNIT_>
struct AnySoftmaxBwd {
  static constexpr int kMaxRegs = 80;
  static constexpr int kKernel = kSoftmaxBwd;
  static constexpr int UNIT = UNIT_;
  using V = V16<DT>;
  using R = AnyRow<DT>;
  using F = AnySoftmaxFwd<DT, UNIT_>;
  static constexpr int EPA = V::EPA;
  static constexpr int NP = EPA / 2;
  struct State {};
  static __device__ __forceinline__ void init(State&) {}
  static __device__ __forceinline__ uint32_t rows_per_group(uint32_t) { return 1u; }  // codes are only read

  // Eq. 9 for the two codes of pair k of a vector (one rounding each, as dequant).
  static __device__ __forceinline__ F2 yhat(uint32_t bits, int k, F2 s2, F2 mn2) {
    return f2_fma(f2_pack((float)((bits >> (8 * k)) & 0xFu), (float)((bits >> (8 * k + 4)) & 0xFu)), s2, mn2);
  }

  static __device__ __forceinline__ void group(Unit<UNIT_>& u, State&, const StagePtrs& p, float*, uint32_t r,
                                               bool active, uint32_t L) {
    if (UNIT_ >= 32 && !active) return;
    R g;
    g.set(active ? r : 0u, L);
    const int ul = u.ul;
    const F2 mn2 = f2_both(active ? p.meta[2 * r] : 0.0f), s2 = f2_both(active ? p.meta[2 * r + 1] : 0.0f);
    F2 dot2 = f2_both(0.0f);
    any_row_vectors<DT, UNIT_>(g, ul, active, [&](uint32_t j, uint32_t msk, auto interior) {
      F2 gv[NP];
      F::pairs_of(*(const typename V::Raw*)(p.data + j * 16u), gv);
      const uint32_t bits = V::load_codes(p.codes, j);
#pragma unroll
      for (int k = 0; k < NP; ++k) {
        const F2 gk = decltype(interior)::value ? gv[k] : F::masked(gv[k], msk, k, 0.0f);
        dot2 = f2_fma(gk, yhat(bits, k, s2, mn2), dot2);
      }
    });
    float d0, d1;
    f2_unpack(dot2, d0, d1);
    const F2 dotv = f2_both(u.template reduce<kOpSum>(d0 + d1));
    any_row_vectors<DT, UNIT_>(g, ul, active, [&](uint32_t j, uint32_t msk, auto interior) {
      F2 gv[NP];
      F::pairs_of(*(const typename V::Raw*)(p.data + j * 16u), gv);
      const uint32_t bits = V::load_codes(p.codes, j);
#pragma unroll
      for (int k = 0; k < NP; ++k) gv[k] = f2_mul(yhat(bits, k, s2, mn2), f2_sub(gv[k], dotv));
      typename V::Raw ow;
      if constexpr (DT == kBF16) {
        ow = make_uint4(f2_to_bf16x2(gv[0]), f2_to_bf16x2(gv[1]), f2_to_bf16x2(gv[2]), f2_to_bf16x2(gv[3]));
      } else {
        float a, b, c, d;
        f2_unpack(gv[0], a, b);
        f2_unpack(gv[1], c, d);
        ow = make_float4(a, b, c, d);
      }
      if constexpr (decltype(interior)::value) *(typename V::Raw*)(p.data + j * 16u) = ow;
      else R::store(p.data, j, ow, msk);
    });
    if (UNIT_ < 32) u.sync();
  }
};

// The any-length softmax at 2 and 8 bits per code.  A 16-byte vector still owns whole code
// bytes (8 or 4 elements times NBITS is a multiple of 8), so interior vectors store their
// codes in one access; on a row's first and last vector the row's bits are merged into
// their bytes, atomically where a byte is shared with a neighbouring row (2 bits: up to
// four rows meet in one byte when the length is odd), so rows need no particular order.
template <int DT, int UNIT_, int NBITS>
struct AnySoftmaxFwdBits {
  static_assert(NBITS == 2 || NBITS == 8, "4 bits have kernels of their own");
  static constexpr int kMaxRegs = 80;
  static constexpr int kKernel = kSoftmaxFwd;
  static constexpr int UNIT = UNIT_;
  using V = V16<DT>;
  using R = AnyRow<DT>;
  using C = CodeIo<DT, NBITS>;
  static constexpr int EPA = V::EPA;
  static constexpr int kVPW = C::BYTES >= 4 ? 1 : 4 / C::BYTES;  // vectors per 32-bit word of codes
  struct State {};
  static __device__ __forceinline__ void init(State&) {}
  static __device__ __forceinline__ uint32_t rows_per_group(uint32_t) { return 1u; }
  static __device__ __forceinline__ float ex(float x, float m, float nm) {
    constexpr float kLog2e = 1.4426950408889634f;
    return DT == kBF16 ? ex2_approx(fmaf(x, kLog2e, nm)) : exp_eval<DT>(x - m);
  }

  static __device__ __forceinline__ void row(Unit<UNIT_>& u, const StagePtrs& p, uint32_t r, bool active, uint32_t L) {
    R g;
    g.set(r, L);
    const int ul = u.ul;
    float m = -INFINITY;
    typename V::MinMax pm;
    pm.init();
    any_row_vectors<DT, UNIT_, kVPW>(g, ul, active, [&](uint32_t j, uint32_t msk, auto interior) {
      const typename V::Raw raw = *(const typename V::Raw*)(p.data + j * 16u);
      if constexpr (decltype(interior)::value) {
        pm.add(raw);
      } else {
        float v[EPA];
        V::widen(raw, v);
#pragma unroll
        for (int k = 0; k < EPA; ++k) m = fmaxf(m, (msk >> k & 1u) ? v[k] : -INFINITY);
      }
    });
    m = u.template reduce<kOpMax>(fmaxf(m, pm.hi()));
    if (!active) m = 0.0f;
    const float nm = -m * 1.4426950408889634f;
    float z = 0.0f;
    any_row_vectors<DT, UNIT_, kVPW>(g, ul, active, [&](uint32_t j, uint32_t msk, auto interior) {
      float v[EPA];
      V::widen(*(const typename V::Raw*)(p.data + j * 16u), v);
#pragma unroll
      for (int k = 0; k < EPA; ++k) {
        const float e = ex(v[k], m, nm);
        if constexpr (decltype(interior)::value) z += e;
        else z += (msk >> k & 1u) ? e : 0.0f;
      }
    });
    z = u.template reduce<kOpSum>(z);
    const float rz = __fdiv_rn(1.0f, active ? z : 1.0f);
    float mn = INFINITY, mx = -INFINITY;
    typename V::MinMax py;
    py.init();
    any_row_vectors<DT, UNIT_, kVPW>(g, ul, active, [&](uint32_t j, uint32_t msk, auto interior) {
      float v[EPA];
      V::widen(*(const typename V::Raw*)(p.data + j * 16u), v);
#pragma unroll
      for (int k = 0; k < EPA; ++k) v[k] = ex(v[k], m, nm) * rz;
      const typename V::Raw yw = V::narrow(v);  // v now holds y as written
      if constexpr (decltype(interior)::value) {
        *(typename V::Raw*)(p.data + j * 16u) = yw;
        py.add(yw);
      } else {
        R::store(p.data, j, yw, msk);
#pragma unroll
        for (int k = 0; k < EPA; ++k) {
          mn = fminf(mn, (msk >> k & 1u) ? v[k] : INFINITY);
          mx = fmaxf(mx, (msk >> k & 1u) ? v[k] : -INFINITY);
        }
      }
    });
    mn = u.template reduce<kOpMin>(fminf(mn, py.lo()));
    mx = u.template reduce<kOpMax>(fmaxf(mx, py.hi()));
    const QRange q = make_qrange(mn, mx, (float)((1 << NBITS) - 1));
    if (active && ul == 0) { p.meta[2 * r] = q.mn; p.meta[2 * r + 1] = q.s; }
    any_row_vectors<DT, UNIT_, kVPW>(g, ul, active, [&](uint32_t j, uint32_t msk, auto interior) {
      float v[EPA];
      V::widen(*(const typename V::Raw*)(p.data + j * 16u), v);
      CodePackerBits<EPA, NBITS> pk;
      pk.init();
      if constexpr (decltype(interior)::value) {
#pragma unroll
        for (int k = 0; k < EPA; ++k) pk.add(k, v[k], q);
        C::store(p.codes, j, pk.acc);
      } else {
#pragma unroll
        for (int k = 0; k < EPA; ++k) pk.add(k, (msk >> k & 1u) ? v[k] : q.mn, q);
        any_merge_codes<NBITS, EPA>(p.codes, j, pk.acc, msk);
      }
    });
  }

  static __device__ __forceinline__ void group(Unit<UNIT_>& u, State&, const StagePtrs& p, float*, uint32_t grp,
                                               bool active, uint32_t L) {
    if (UNIT_ >= 32 && !active) return;
    row(u, p, active ? grp : 0u, active, L);
    if (UNIT_ < 32) u.sync();
  }
};

template <int DT, int UNIT_, int NBITS>
struct AnySoftmaxBwdBits {
  static_assert(NBITS == 2 || NBITS == 8, "4 bits have kernels of their own");
  static constexpr int kMaxRegs = 80;
  static constexpr int kKernel = kSoftmaxBwd;
  static constexpr int UNIT = UNIT_;
  using V = V16<DT>;
  using R = AnyRow<DT>;
  using C = CodeIo<DT, NBITS>;
  static constexpr int EPA = V::EPA;
  struct State {};
  static __device__ __forceinline__ void init(State&) {}
  static __device__ __forceinline__ uint32_t rows_per_group(uint32_t) { return 1u; }  // codes are only read

  static __device__ __forceinline__ float yhat(const uint32_t* w, int k, float mn, float s) {
    constexpr int PER = 32 / NBITS;
    return dequant((w[k / PER] >> (NBITS * (k % PER))) & ((1u << NBITS) - 1u), mn, s);
  }

  static __device__ __forceinline__ void group(Unit<UNIT_>& u, State&, const StagePtrs& p, float*, uint32_t r,
                                               bool active, uint32_t L) {
    if (UNIT_ >= 32 && !active) return;
    R g;
    g.set(active ? r : 0u, L);
    const int ul = u.ul;
    const float mn = active ? p.meta[2 * r] : 0.0f;
    const float s = active ? p.meta[2 * r + 1] : 0.0f;
    float dot = 0.0f;
    any_row_vectors<DT, UNIT_>(g, ul, active, [&](uint32_t j, uint32_t msk, auto interior) {
      float v[EPA];
      V::widen(*(const typename V::Raw*)(p.data + j * 16u), v);
      uint32_t w[C::W];
      C::load(p.codes, j, w);
#pragma unroll
      for (int k = 0; k < EPA; ++k) {
        const float yh = yhat(w, k, mn, s);
        if constexpr (decltype(interior)::value) dot = fmaf(v[k], yh, dot);
        else dot = fmaf((msk >> k & 1u) ? v[k] : 0.0f, yh, dot);
      }
    });
    dot = u.template reduce<kOpSum>(dot);
    any_row_vectors<DT, UNIT_>(g, ul, active, [&](uint32_t j, uint32_t msk, auto interior) {
      float v[EPA];
      V::widen(*(const typename V::Raw*)(p.data + j * 16u), v);
      uint32_t w[C::W];
      C::load(p.codes, j, w);
#pragma unroll
      for (int k = 0; k < EPA; ++k) v[k] = yhat(w, k, mn, s) * (v[k] - dot);
      const typename V::Raw ow = V::narrow(v);
      if constexpr (decltype(interior)::value) *(typename V::Raw*)(p.data + j * 16u) = ow;
      else R::store(p.data, j, ow, msk);
    });
    if (UNIT_ < 32) u.sync();
  }
};

// ---------------------------------------------------------------- odd rows, fixed length
// Softmax rows of a compile-time length that is not a whole number of 16-byte vectors (the
// attention widths 197 and 257, and 49, 50, 145, 196, 198, 577, 1025).  Rows are read as 2-element
// words on the tile's even-element grid.  With an odd length a row that starts on an even
// element shares its LAST word (and code byte) with the next row, a row that starts on an
// odd element shares its FIRST word with the previous one; a unit handles such a pair back
// to back.  With the length fixed every mask is resolved at compile time except on the one
// or two words that are actually shared or ragged.  HP names a row's kind: 0 starts even
// and shares its last word, 1 starts odd and shares its first, 2 (even lengths) shares
// nothing.
template <int DT> struct P2;
template <> struct P2<kBF16> {
  using Raw = uint32_t;
  static constexpr int kWordBytes = 4;
  static __device__ __forceinline__ Raw load(const unsigned char* d, uint32_t a) { return *(const uint32_t*)(d + a * 4u); }
  static __device__ __forceinline__ float lo(Raw w) { return __uint_as_float(w << 16); }
  static __device__ __forceinline__ float hi(Raw w) { return __uint_as_float(w & 0xffff0000u); }
  static __device__ __forceinline__ Raw pack(float a, float b) {
    __nv_bfloat162 t = __floats2bfloat162_rn(a, b);
    return *(uint32_t*)&t;
  }
  static __device__ __forceinline__ void store(unsigned char* d, uint32_t a, Raw w) { *(uint32_t*)(d + a * 4u) = w; }
  static __device__ __forceinline__ void store_lo(unsigned char* d, uint32_t a, Raw w) { *(uint16_t*)(d + a * 4u) = (uint16_t)w; }
  static __device__ __forceinline__ void store_hi(unsigned char* d, uint32_t a, Raw w) { *(uint16_t*)(d + a * 4u + 2) = (uint16_t)(w >> 16); }
};
template <> struct P2<kF32> {
  using Raw = float2;
  static constexpr int kWordBytes = 8;
  static __device__ __forceinline__ Raw load(const unsigned char* d, uint32_t a) { return *(const float2*)(d + a * 8u); }
  static __device__ __forceinline__ float lo(Raw w) { return w.x; }
  static __device__ __forceinline__ float hi(Raw w) { return w.y; }
  static __device__ __forceinline__ Raw pack(float a, float b) { return make_float2(a, b); }
  static __device__ __forceinline__ void store(unsigned char* d, uint32_t a, Raw w) { *(float2*)(d + a * 8u) = w; }
  static __device__ __forceinline__ void store_lo(unsigned char* d, uint32_t a, Raw w) { *(float*)(d + a * 8u) = w.x; }
  static __device__ __forceinline__ void store_hi(unsigned char* d, uint32_t a, Raw w) { *(float*)(d + a * 8u + 4) = w.y; }
};

template <int UNIT_, int LCT>
struct PairGeom {
  static constexpr bool kOdd = (LCT % 2) == 1;             // even lengths: rows own whole words
  static constexpr int NACC = (LCT + 1) / 2;               // words covering one row
  static constexpr int ITERS = (NACC + UNIT_ - 1) / UNIT_;
  static constexpr int NFULL = NACC / UNIT_;               // iterations in which every lane has a word
  static constexpr int REM = NACC % UNIT_;
  static constexpr int LAST_I = (NACC - 1) / UNIT_;        // where the row's last word sits
  static constexpr int LAST_UL = (NACC - 1) % UNIT_;
  static __device__ __forceinline__ bool has(int i, int ul) { return i < NFULL || ul < REM; }
};

template <int DT, int UNIT_, int LCT>
struct PairSoftmaxFwd {
  static constexpr int kMaxRegs = 96;  // 4 CTAs of 160 threads per SM
  static constexpr int kKernel = kSoftmaxFwd;
  static constexpr int UNIT = UNIT_;
  using P = P2<DT>;
  using G = PairGeom<UNIT_, LCT>;
  struct State {};
  static __device__ __forceinline__ void init(State&) {}
  static __device__ __forceinline__ uint32_t rows_per_group(uint32_t) { return 2u; }

  // HP = 0: the row starts on an even element (high half of its last word is foreign);
  // HP = 1: it starts on an odd element (low half of its first word is foreign).
  template <int HP>
  static __device__ __forceinline__ void row(Unit<UNIT_>& u, const StagePtrs& p, uint32_t r, bool active) {
    const uint32_t a0 = (r * (uint32_t)LCT) >> 1;
    const int ul = u.ul;
    float e[G::ITERS][2];
    float m = -INFINITY;
#pragma unroll
    for (int i = 0; i < G::ITERS; ++i) {
      e[i][0] = -INFINITY;
      e[i][1] = -INFINITY;
      if (active && G::has(i, ul)) {
        const typename P::Raw w = P::load(p.data, a0 + ul + UNIT_ * i);
        e[i][0] = P::lo(w);
        e[i][1] = P::hi(w);
      }
      if (HP == 1 && i == 0 && ul == 0) e[i][0] = -INFINITY;
      if (HP == 0 && i == G::LAST_I && ul == G::LAST_UL) e[i][1] = -INFINITY;
      m = fmaxf(m, fmaxf(e[i][0], e[i][1]));
    }
    m = u.template reduce<kOpMax>(m);
    if (!active) m = 0.0f;
    float z = 0.0f;
#pragma unroll
    for (int i = 0; i < G::ITERS; ++i) {
      e[i][0] = exp_eval<DT>(e[i][0] - m);  // foreign / absent elements: exp(-inf) = 0
      e[i][1] = exp_eval<DT>(e[i][1] - m);
      z += e[i][0] + e[i][1];
    }
    z = u.template reduce<kOpSum>(z);
    const float rz = __fdiv_rn(1.0f, active ? z : 1.0f);
    float mn = INFINITY, mx = -INFINITY;
#pragma unroll
    for (int i = 0; i < G::ITERS; ++i) {
      const typename P::Raw w = P::pack(e[i][0] * rz, e[i][1] * rz);
      e[i][0] = P::lo(w);  // y as written
      e[i][1] = P::hi(w);
      const bool mine = active && G::has(i, ul);
      const bool drop_lo = HP == 1 && i == 0 && ul == 0;
      const bool drop_hi = HP == 0 && i == G::LAST_I && ul == G::LAST_UL;
      if (mine) {
        if (drop_lo) P::store_hi(p.data, a0 + ul + UNIT_ * i, w);
        else if (drop_hi) P::store_lo(p.data, a0 + ul + UNIT_ * i, w);
        else P::store(p.data, a0 + ul + UNIT_ * i, w);
        const float v0 = drop_lo ? e[i][1] : e[i][0], v1 = drop_hi ? e[i][0] : e[i][1];
        mn = fminf(mn, fminf(v0, v1));
        mx = fmaxf(mx, fmaxf(v0, v1));
      }
    }
    mn = u.template reduce<kOpMin>(mn);
    mx = u.template reduce<kOpMax>(mx);
    const QRange q = make_qrange(mn, mx);
    if (active && ul == 0) { p.meta[2 * r] = q.mn; p.meta[2 * r + 1] = q.s; }
#pragma unroll
    for (int i = 0; i < G::ITERS; ++i) {
      if (active && G::has(i, ul)) {
        const bool drop_lo = HP == 1 && i == 0 && ul == 0;
        const bool drop_hi = HP == 0 && i == G::LAST_I && ul == G::LAST_UL;
        CodePacker<2> pk;
        pk.init();
        pk.add(0, drop_lo ? q.mn : e[i][0], q);
        pk.add(1, drop_hi ? q.mn : e[i][1], q);  // a dropped element codes as 0
        uint32_t byte = pk.acc & 0xFFu;
        if (drop_lo) byte |= p.codes[a0 + ul + UNIT_ * i] & 0x0Fu;  // low nibble: the previous row's
        p.codes[a0 + ul + UNIT_ * i] = (unsigned char)byte;
      }
    }
  }

  static __device__ __forceinline__ void group(Unit<UNIT_>& u, State&, const StagePtrs& p, float*, uint32_t grp,
                                               bool active, uint32_t) {
    const uint32_t r = active ? 2 * grp : 0;
    if (G::kOdd) {
      row<0>(u, p, r, active);
      u.sync();  // the odd row reads the shared word and code byte the even row left
      row<1>(u, p, r + 1, active);
    } else {
      row<2>(u, p, r, active);
      row<2>(u, p, r + 1, active);
    }
    u.sync();
  }
};

// bfloat16 form of the forward: maxima and minima are taken on packed bfloat16 pairs,
// and the exponent's argument is one fused multiply-add.
template <int UNIT_, int LCT>
struct PairSoftmaxFwd<kBF16, UNIT_, LCT> {
  // 4 CTAs of 160 threads per SM; width 257 (17 words per lane and row) runs with 3 CTAs of three stages
  // and 128 registers: 28.6 -> 28.0 us (with 96 registers three CTAs had measured slower than four)
  static constexpr int kMaxRegs = LCT == 257 ? 128 : 96;
  static constexpr int kKernel = kSoftmaxFwd;
  static constexpr int UNIT = UNIT_;
  using G = PairGeom<UNIT_, LCT>;
  struct State {};
  static __device__ __forceinline__ void init(State&) {}
  static __device__ __forceinline__ uint32_t rows_per_group(uint32_t) { return 2u; }

  static __device__ __forceinline__ uint32_t max2(uint32_t a, uint32_t b) {
    __nv_bfloat162 r = __hmax2(*(__nv_bfloat162*)&a, *(__nv_bfloat162*)&b);
    return *(uint32_t*)&r;
  }
  static __device__ __forceinline__ uint32_t min2(uint32_t a, uint32_t b) {
    __nv_bfloat162 r = __hmin2(*(__nv_bfloat162*)&a, *(__nv_bfloat162*)&b);
    return *(uint32_t*)&r;
  }
  static __device__ __forceinline__ float lo(uint32_t w) { return __uint_as_float(w << 16); }
  static __device__ __forceinline__ float hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }

  // The two rows of a pair are worked on TOGETHER, phase by phase, so that each row's
  // shuffle and special-function latencies hide behind the other row's arithmetic.  HP = 0
  // is the row that starts on an even element (the high half of its last word is the next
  // row's), HP = 1 the one that starts on an odd element (the low half of its first word is
  // the previous row's).  An inactive unit (no pair left in this round) runs on rows 0 and 1
  // and stores nothing, so that every lane takes part in the shuffles.
  struct Regs {
    uint32_t w[G::ITERS];      // input words, later y as written
    F2 e[G::ITERS];            // the two exponentials of each word, as a packed binary32 pair
  };
  template <int HP>
  static __device__ __forceinline__ bool drop_lo(int i, int ul) { return HP == 1 && i == 0 && ul == 0; }
  template <int HP>
  static __device__ __forceinline__ bool drop_hi(int i, int ul) { return HP == 0 && i == G::LAST_I && ul == G::LAST_UL; }

  // Loads the row's words (foreign and absent halves become -inf, so that they vanish from the
  // exponentials) and returns the row's largest AND smallest input: softmax is monotone, so the
  // extreme outputs sit at the extreme inputs and the range of y needs no reduction of its own
  // (see front()).
  template <int HP>
  static __device__ __forceinline__ void load_minmax(Regs& R, const uint32_t* words, int ul, float& mx, float& mn) {
    constexpr uint32_t kNegInf2 = 0xFF80FF80u, kPosInf2 = 0x7F807F80u;
    uint32_t mx2 = kNegInf2, mn2 = kPosInf2;
#pragma unroll
    for (int i = 0; i < G::ITERS; ++i) {
      uint32_t w = kNegInf2, wn = kPosInf2;
      if (G::has(i, ul)) {
        w = words[UNIT_ * i];
        wn = w;
      }
      if (drop_lo<HP>(i, ul)) {  // foreign low half
        w = (w & 0xffff0000u) | 0xFF80u;
        wn = (wn & 0xffff0000u) | 0x7F80u;
      }
      if (drop_hi<HP>(i, ul)) {  // foreign high half
        w = (w & 0x0000ffffu) | 0xFF800000u;
        wn = (wn & 0x0000ffffu) | 0x7F800000u;
      }
      R.w[i] = w;
      mx2 = max2(mx2, w);
      mn2 = min2(mn2, wn);
    }
    mx = fmaxf(lo(mx2), hi(mx2));
    mn = fminf(lo(mn2), hi(mn2));
  }

  // All binary32 arithmetic below runs on packed pairs (one instruction per word).
  static __device__ __forceinline__ float exp_sum(Regs& R, float nm) {  // nm = -(row maximum) * log2 e
    constexpr float kLog2e = 1.4426950408889634f;
    const F2 k2 = f2_both(kLog2e), nm2 = f2_both(nm);
    F2 z2 = f2_both(0.0f);
#pragma unroll
    for (int i = 0; i < G::ITERS; ++i) {
      float a0, a1;
      f2_unpack(f2_fma(f2_from_bf16x2(R.w[i]), k2, nm2), a0, a1);
      R.e[i] = f2_pack(ex2_approx(a0), ex2_approx(a1));  // foreign / absent: 2^-inf = 0
      z2 = f2_add(z2, R.e[i]);
    }
    float z0, z1;
    f2_unpack(z2, z0, z1);
    return z0 + z1;
  }

  template <int HP>
  static __device__ __forceinline__ void scale_store(Regs& R, float rz, uint32_t* out, int ul, bool active) {
    const F2 rz2 = f2_both(rz);
#pragma unroll
    for (int i = 0; i < G::ITERS; ++i) {
      const uint32_t w = f2_to_bf16x2(f2_mul(R.e[i], rz2));  // y as written
      R.w[i] = w;
      if (active && G::has(i, ul)) {
        if (drop_lo<HP>(i, ul)) *((uint16_t*)(out + UNIT_ * i) + 1) = (uint16_t)(w >> 16);
        else if (drop_hi<HP>(i, ul)) *(uint16_t*)(out + UNIT_ * i) = (uint16_t)w;
        else out[UNIT_ * i] = w;
      }
    }
  }

  // y as written at the row's smallest and largest input -- the very operations every element
  // goes through (one fused multiply-add, 2^x, the scaling, the rounding to bfloat16), each of
  // them monotone, so these ARE the minimum and the maximum of the row's y as written.
  static __device__ __forceinline__ void range_of_y(float x_min, float x_max, float nm, float rz, float& mn, float& mx) {
    float a0, a1;
    f2_unpack(f2_fma(f2_pack(x_min, x_max), f2_both(1.4426950408889634f), f2_both(nm)), a0, a1);
    const uint32_t w = f2_to_bf16x2(f2_mul(f2_pack(ex2_approx(a0), ex2_approx(a1)), f2_both(rz)));
    mn = lo(w);
    mx = hi(w);
  }

  // Code byte of word i of a row (a foreign half codes as 0: it is replaced by the minimum).
  template <int HP>
  static __device__ __forceinline__ uint32_t code_byte(const Regs& R, int i, int ul, const QRange& q, F2 min2, F2 inv2) {
    float v0 = lo(R.w[i]), v1 = hi(R.w[i]);
    if (drop_lo<HP>(i, ul)) v0 = q.mn;
    if (drop_hi<HP>(i, ul)) v1 = q.mn;
    return f2_code_byte(f2_pack(v0, v1), min2, inv2) & 0xFFu;
  }

  // Everything up to the quantiser ranges of the pair's two rows (rows r and r + 1): y is
  // written, A.w / B.w hold y as written, the metadata is stored.  LEVELS = 2^N - 1 of Eq. 8.
  template <int LEVELS>
  static __device__ __forceinline__ void front(Unit<UNIT_>& u, const StagePtrs& p, uint32_t r, bool active, Regs& A,
                                               Regs& B, QRange& qA, QRange& qB) {
    const int ul = u.ul;
    const uint32_t a0 = (r * (uint32_t)LCT) >> 1, a1 = ((r + 1) * (uint32_t)LCT) >> 1;  // odd: a1 = a0 + NACC - 1
    constexpr int HA = G::kOdd ? 0 : 2, HB = G::kOdd ? 1 : 2;  // the kinds of the pair's two rows
    float mA, mB, nA, nB;  // the rows' largest and smallest inputs
    load_minmax<HA>(A, (const uint32_t*)p.data + a0 + ul, ul, mA, nA);
    load_minmax<HB>(B, (const uint32_t*)p.data + a1 + ul, ul, mB, nB);
    {
      // all four are bfloat16 values: the maxima travel down one shuffle chain as a packed pair,
      // the minima down another
      __nv_bfloat162 pm = __floats2bfloat162_rn(mA, mB), pn = __floats2bfloat162_rn(nA, nB);
      uint32_t w = *(uint32_t*)&pm, v = *(uint32_t*)&pn;
#pragma unroll
      for (int o = UNIT_ / 2; o > 0; o >>= 1) {
        w = max2(w, __shfl_xor_sync(0xffffffffu, w, o));
        v = min2(v, __shfl_xor_sync(0xffffffffu, v, o));
      }
      mA = lo(w);
      mB = hi(w);
      nA = lo(v);
      nB = hi(v);
    }
    constexpr float kLog2e = 1.4426950408889634f;
    const float nmA = -mA * kLog2e, nmB = -mB * kLog2e;
    float zA = exp_sum(A, nmA);
    float zB = exp_sum(B, nmB);
    {
      F2 z2 = f2_pack(zA, zB);  // the two sums are reduced together, one packed addition per step
#pragma unroll
      for (int o = UNIT_ / 2; o > 0; o >>= 1) {
        float x0, x1;
        f2_unpack(z2, x0, x1);
        z2 = f2_add(z2, f2_pack(__shfl_xor_sync(0xffffffffu, x0, o), __shfl_xor_sync(0xffffffffu, x1, o)));
      }
      f2_unpack(z2, zA, zB);
    }
    // 1 / z to about an ulp (hardware reciprocal and one correction step): y is rounded to 8 bits
    const float rA0 = rcp_approx(zA), rB0 = rcp_approx(zB);
    const float rzA = __fmaf_rn(__fmaf_rn(-zA, rA0, 1.0f), rA0, rA0), rzB = __fmaf_rn(__fmaf_rn(-zB, rB0, 1.0f), rB0, rB0);
    scale_store<HA>(A, rzA, (uint32_t*)p.data + a0 + ul, ul, active);
    scale_store<HB>(B, rzB, (uint32_t*)p.data + a1 + ul, ul, active);
    float mnA, mxA, mnB, mxB;
    range_of_y(nA, mA, nmA, rzA, mnA, mxA);
    range_of_y(nB, mB, nmB, rzB, mnB, mxB);
    // Eq. 8's two correctly rounded quotients per row, LEVELS / d and d / LEVELS, for both rows with ONE
    // division: lane 0 of the unit forms LEVELS / dA, lane 1 dA / LEVELS, lane 2 LEVELS / dB, lane 3 dB / LEVELS
    // (the other lanes repeat them), and four shuffles hand the results round.
    {
      const float dA = __fsub_rn(mxA, mnA), dB = __fsub_rn(mxB, mnB);
      const float d = (ul & 2) ? dB : dA;
      const bool odd = (ul & 1) != 0;
      float quo = __fdiv_rn(odd ? d : (float)LEVELS, odd ? (float)LEVELS : d);
      if (d == 0.0f) quo = 0.0f;  // a constant row: inv = s = 0
      const int base = threadIdx.x & 31 & ~(UNIT_ - 1);
      qA.mn = mnA;
      qB.mn = mnB;
      qA.inv = __shfl_sync(0xffffffffu, quo, base);
      qA.s = __shfl_sync(0xffffffffu, quo, base + 1);
      qB.inv = __shfl_sync(0xffffffffu, quo, base + 2);
      qB.s = __shfl_sync(0xffffffffu, quo, base + 3);
    }
    if (active && ul == 0) {
      p.meta[2 * r] = qA.mn; p.meta[2 * r + 1] = qA.s;
      p.meta[2 * r + 2] = qB.mn; p.meta[2 * r + 3] = qB.s;
    }
  }

  static __device__ __forceinline__ void group(Unit<UNIT_>& u, State&, const StagePtrs& p, float*, uint32_t grp,
                                               bool active, uint32_t) {
    const uint32_t r = active ? 2 * grp : 0;
    const int ul = u.ul;
    const uint32_t a0 = (r * (uint32_t)LCT) >> 1, a1 = ((r + 1) * (uint32_t)LCT) >> 1;
    Regs A, B;
    QRange qA, qB;
    constexpr int HA = G::kOdd ? 0 : 2, HB = G::kOdd ? 1 : 2;  // the kinds of the pair's two rows
    front<15>(u, p, r, active, A, B, qA, qB);
    // The byte the two rows share: row A's last element is its low nibble, row B's first
    // its high nibble.  A's nibble travels by shuffle to the lane that owns B's first word.
    const F2 minA = f2_both(qA.mn), invA = f2_both(qA.inv), minB = f2_both(qB.mn), invB = f2_both(qB.inv);
    const uint32_t a_last = code_byte<HA>(A, G::LAST_I, ul, qA, minA, invA);
    const uint32_t shared_lo = __shfl_sync(0xffffffffu, a_last, (threadIdx.x & 31 & ~(UNIT_ - 1)) | G::LAST_UL);
    unsigned char* cA = p.codes + a0 + ul;
    unsigned char* cB = p.codes + a1 + ul;
#pragma unroll
    for (int i = 0; i < G::ITERS; ++i) {
      if (active && G::has(i, ul)) {
        if (!G::kOdd || !(i == G::LAST_I && ul == G::LAST_UL))
          cA[UNIT_ * i] = (unsigned char)code_byte<HA>(A, i, ul, qA, minA, invA);
        uint32_t b = code_byte<HB>(B, i, ul, qB, minB, invB);
        if (G::kOdd && i == 0 && ul == 0) b |= shared_lo & 0x0Fu;
        cB[UNIT_ * i] = (unsigned char)b;
      }
    }
    u.sync();  // orders this pair's shared-memory writes before the unit's next pair
  }
};

template <int DT, int UNIT_, int LCT>
struct PairSoftmaxBwd {
  // 4 CTAs of 160 threads per SM; the bfloat16 kernel at width 257 runs with 3 CTAs per SM (its stages
  // fit a quarter of the shared memory only twice) and may use the registers that frees: 25.5 -> 24.9 us
  static constexpr int kMaxRegs = (LCT == 257 && DT == kBF16) ? 128 : 96;
  static constexpr int kKernel = kSoftmaxBwd;
  static constexpr int UNIT = UNIT_;
  using P = P2<DT>;
  using G = PairGeom<UNIT_, LCT>;
  struct State {};
  static __device__ __forceinline__ void init(State&) {}
  static __device__ __forceinline__ uint32_t rows_per_group(uint32_t) { return 2u; }

  // An inactive unit runs on row 0 and stores nothing (see the forward).
  template <int HP>
  static __device__ __forceinline__ void row(Unit<UNIT_>& u, const StagePtrs& p, uint32_t r, bool active) {
    const uint32_t a0 = (r * (uint32_t)LCT) >> 1;
    const int ul = u.ul;
    const float mn = p.meta[2 * r];
    const float s = p.meta[2 * r + 1];
    float g[G::ITERS][2], yh[G::ITERS][2];
    float dot = 0.0f;
#pragma unroll
    for (int i = 0; i < G::ITERS; ++i) {
      if (G::has(i, ul)) {
        const typename P::Raw w = P::load(p.data, a0 + ul + UNIT_ * i);
        const uint32_t b = p.codes[a0 + ul + UNIT_ * i];
        g[i][0] = P::lo(w);
        g[i][1] = P::hi(w);
        yh[i][0] = dequant(b & 0xFu, mn, s);
        yh[i][1] = dequant(b >> 4, mn, s);
      } else {
        g[i][0] = 0.0f; g[i][1] = 0.0f; yh[i][0] = 0.0f; yh[i][1] = 0.0f;
      }
      if (HP == 1 && i == 0 && ul == 0) g[i][0] = 0.0f;
      if (HP == 0 && i == G::LAST_I && ul == G::LAST_UL) g[i][1] = 0.0f;
      dot = fmaf(g[i][0], yh[i][0], dot);
      dot = fmaf(g[i][1], yh[i][1], dot);
    }
    dot = u.template reduce<kOpSum>(dot);
#pragma unroll
    for (int i = 0; i < G::ITERS; ++i) {
      if (active && G::has(i, ul)) {
        const typename P::Raw w = P::pack(yh[i][0] * (g[i][0] - dot), yh[i][1] * (g[i][1] - dot));
        const bool drop_lo = HP == 1 && i == 0 && ul == 0;
        const bool drop_hi = HP == 0 && i == G::LAST_I && ul == G::LAST_UL;
        if (drop_lo) P::store_hi(p.data, a0 + ul + UNIT_ * i, w);
        else if (drop_hi) P::store_lo(p.data, a0 + ul + UNIT_ * i, w);
        else P::store(p.data, a0 + ul + UNIT_ * i, w);
      }
    }
  }

  static __device__ __forceinline__ void group(Unit<UNIT_>& u, State&, const StagePtrs& p, float*, uint32_t grp,
                                               bool active, uint32_t) {
    const uint32_t r = active ? 2 * grp : 0;
    if (G::kOdd) {
      row<0>(u, p, r, active);
      u.sync();  // the odd row's first word holds the even row's last result
      row<1>(u, p, r + 1, active);
    } else {
      row<2>(u, p, r, active);
      row<2>(u, p, r + 1, active);
    }
    u.sync();
  }
};

// ---------------------------------------------------------------- fixed widths at 2 and 8 bits
// The attention widths 197 and 257 with Eq. 8 at N = 2 or N = 8.  Rows are read as 2-element
// words like the 4-bit fixed-width kernels, one row at a time per 8-lane unit.  At 8 bits an
// element owns a whole code byte, so no byte is ever shared.  At 2 bits four elements share a
// byte and a row of odd length shares bytes with both neighbours -- but EIGHT consecutive rows
// always own whole bytes (16 L bits).  The four units of a warp take four consecutive row
// pairs, write one UNPACKED code byte per element into a scratch area of the CTA, and the warp
// then packs its own eight rows, four scratch bytes to a code byte: nothing is merged
// atomically and no warp waits for another.
template <int DT, int UNIT_, int LCT, int NBITS>
struct PairSoftmaxFwdBits {
  static_assert(NBITS == 2 || NBITS == 8, "4 bits have kernels of their own");
  static constexpr int kMaxRegs = 96;
  static constexpr int kKernel = kSoftmaxFwd;
  static constexpr int UNIT = UNIT_;
  static_assert(UNIT_ == 8, "four units per warp: eight consecutive rows per warp and round");
  static constexpr int kTabFloats = 0;            // `tab` is the CTA's scratch area itself, not a per-unit table
  using P = P2<DT>;
  using G = PairGeom<UNIT_, LCT>;
  struct State {};
  static __device__ __forceinline__ void init(State&) {}
  static __device__ __forceinline__ uint32_t rows_per_group(uint32_t) { return 2u; }

  // bytes: where this row's unpacked codes go (element e of the tile at bytes[e]): the code
  // area itself at 8 bits, the CTA's scratch at 2 bits.
  template <int HP>
  static __device__ __forceinline__ void row(Unit<UNIT_>& u, const StagePtrs& p, unsigned char* bytes, uint32_t r,
                                             bool active) {
    const uint32_t a0 = (r * (uint32_t)LCT) >> 1;
    const int ul = u.ul;
    F2 e[G::ITERS];
    float m = -INFINITY;
#pragma unroll
    for (int i = 0; i < G::ITERS; ++i) {
      float v0 = -INFINITY, v1 = -INFINITY;
      if (active && G::has(i, ul)) {
        const typename P::Raw w = P::load(p.data, a0 + ul + UNIT_ * i);
        v0 = P::lo(w);
        v1 = P::hi(w);
      }
      if (HP == 1 && i == 0 && ul == 0) v0 = -INFINITY;                        // the previous row's element
      if (HP == 0 && i == G::LAST_I && ul == G::LAST_UL) v1 = -INFINITY;      // the next row's element
      e[i] = f2_pack(v0, v1);
      m = fmaxf(m, fmaxf(v0, v1));
    }
    m = u.template reduce<kOpMax>(m);
    if (!active) m = 0.0f;
    constexpr float kLog2e = 1.4426950408889634f;
    const F2 k2 = f2_both(kLog2e), c2 = f2_both(DT == kBF16 ? -m * kLog2e : m);
    F2 z2 = f2_both(0.0f);
#pragma unroll
    for (int i = 0; i < G::ITERS; ++i) {
      float a, b;
      f2_unpack(DT == kBF16 ? f2_fma(e[i], k2, c2) : f2_mul(k2, f2_sub(e[i], c2)), a, b);
      e[i] = f2_pack(ex2_approx(a), ex2_approx(b));  // foreign / absent elements: 2^-inf = 0
      z2 = f2_add(z2, e[i]);
    }
    float z0, z1;
    f2_unpack(z2, z0, z1);
    const float z = u.template reduce<kOpSum>(z0 + z1);
    const float zz = active ? z : 1.0f;
    float rz;
    if constexpr (DT == kBF16) {
      const float ra = rcp_approx(zz);  // about an ulp after the correction step; y keeps 8 bits
      rz = __fmaf_rn(__fmaf_rn(-zz, ra, 1.0f), ra, ra);
    } else {
      rz = __fdiv_rn(1.0f, zz);
    }
    const F2 rz2 = f2_both(rz);
    float mn = INFINITY, mx = -INFINITY;
#pragma unroll
    for (int i = 0; i < G::ITERS; ++i) {
      float y0, y1;
      f2_unpack(f2_mul(e[i], rz2), y0, y1);
      const typename P::Raw w = P::pack(y0, y1);
      y0 = P::lo(w);  // y as written
      y1 = P::hi(w);
      e[i] = f2_pack(y0, y1);
      if (active && G::has(i, ul)) {
        const bool drop_lo = HP == 1 && i == 0 && ul == 0;
        const bool drop_hi = HP == 0 && i == G::LAST_I && ul == G::LAST_UL;
        if (drop_lo) P::store_hi(p.data, a0 + ul + UNIT_ * i, w);
        else if (drop_hi) P::store_lo(p.data, a0 + ul + UNIT_ * i, w);
        else P::store(p.data, a0 + ul + UNIT_ * i, w);
        const float v0 = drop_lo ? y1 : y0, v1 = drop_hi ? y0 : y1;
        mn = fminf(mn, fminf(v0, v1));
        mx = fmaxf(mx, fmaxf(v0, v1));
      }
    }
    mn = u.template reduce<kOpMin>(mn);
    mx = u.template reduce<kOpMax>(mx);
    const QRange q = make_qrange(mn, mx, (float)((1 << NBITS) - 1));
    if (active && ul == 0) { p.meta[2 * r] = q.mn; p.meta[2 * r + 1] = q.s; }
    const F2 min2 = f2_both(q.mn), inv2 = f2_both(q.inv), magic2 = f2_both(12582912.0f);
    constexpr uint32_t kMask = (1u << NBITS) - 1u;
#pragma unroll
    for (int i = 0; i < G::ITERS; ++i) {
      if (active && G::has(i, ul)) {
        const bool drop_lo = HP == 1 && i == 0 && ul == 0;
        const bool drop_hi = HP == 0 && i == G::LAST_I && ul == G::LAST_UL;
        float t0, t1;
        f2_unpack(f2_add(f2_scaled(e[i], min2, inv2), magic2), t0, t1);
        const uint32_t c0 = __float_as_uint(t0) & kMask, c1 = __float_as_uint(t1) & kMask;
        unsigned char* dst = bytes + 2u * (a0 + ul + UNIT_ * i);
        if (drop_lo) dst[1] = (unsigned char)c1;
        else if (drop_hi) dst[0] = (unsigned char)c0;
        else *(uint16_t*)dst = (uint16_t)(c0 | (c1 << 8));
      }
    }
  }

  static __device__ __forceinline__ void group(Unit<UNIT_>& u, State&, const StagePtrs& p, float* tab, uint32_t grp,
                                               bool active, uint32_t) {
    const uint32_t r = active ? 2 * grp : 0;
    unsigned char* bytes = NBITS == 8 ? p.codes : (unsigned char*)tab;
    if (G::kOdd) {
      row<0>(u, p, bytes, r, active);
      u.sync();  // the odd row reads the word it shares with the even row
      row<1>(u, p, bytes, r + 1, active);
    } else {
      row<2>(u, p, bytes, r, active);
      row<2>(u, p, bytes, r + 1, active);
    }
    u.sync();
    if (NBITS == 2) {
      // The warp's four units hold four consecutive pairs (the planner leaves the units unspread
      // and gives a tile a multiple of four pairs): rows 2 g0 .. 2 g0 + 7, whole code bytes.
      __syncwarp();
      const uint32_t e_begin = (grp - (uint32_t)(u.uid & 3)) * 2u * (uint32_t)LCT;
      if (active) {
        // eight scratch bytes (8-byte aligned: e_begin is a multiple of 8 L) make two code bytes
        for (uint32_t b = threadIdx.x & 31u; b < (uint32_t)LCT; b += 32u) {
          const uint2 w = *(const uint2*)(bytes + e_begin + 8u * b);
          const uint32_t lo = (w.x & 3u) | ((w.x >> 6) & 0xCu) | ((w.x >> 12) & 0x30u) | ((w.x >> 18) & 0xC0u);
          const uint32_t hi = (w.y & 3u) | ((w.y >> 6) & 0xCu) | ((w.y >> 12) & 0x30u) | ((w.y >> 18) & 0xC0u);
          *(uint16_t*)(p.codes + e_begin / 4u + 2u * b) = (uint16_t)(lo | (hi << 8));
        }
      }
      __syncwarp();  // the scratch bytes are free again for the warp's next round
    }
  }
};

// bfloat16 form of the forward at 2 and 8 bits: the two rows of a pair are worked on together
// by the 4-bit kernel's own front part (packed arithmetic, shared shuffle chains, one division);
// only the code phase differs -- a byte per element into the code area (8 bits), or a nibble per
// 2-element word into the scratch that the warp then packs (2 bits).
template <int UNIT_, int LCT, int NBITS>
struct PairSoftmaxFwdBits<kBF16, UNIT_, LCT, NBITS> {
  static_assert(NBITS == 2 || NBITS == 8, "4 bits have kernels of their own");
  static_assert(UNIT_ == 8, "four units per warp: eight consecutive rows per warp and round");
  using B4 = PairSoftmaxFwd<kBF16, UNIT_, LCT>;
  using G = PairGeom<UNIT_, LCT>;
  static constexpr int kMaxRegs = 96;
  static constexpr int kKernel = kSoftmaxFwd;
  static constexpr int UNIT = UNIT_;
  static constexpr int kTabFloats = 0;  // `tab` is the CTA's scratch area itself, not a per-unit table
  struct State {};
  static __device__ __forceinline__ void init(State&) {}
  static __device__ __forceinline__ uint32_t rows_per_group(uint32_t) { return 2u; }

  static __device__ __forceinline__ void group(Unit<UNIT_>& u, State&, const StagePtrs& p, float* tab, uint32_t grp,
                                               bool active, uint32_t) {
    const uint32_t r = active ? 2 * grp : 0;
    const int ul = u.ul;
    const uint32_t a0 = (r * (uint32_t)LCT) >> 1, a1 = ((r + 1) * (uint32_t)LCT) >> 1;
    typename B4::Regs A, B;
    QRange qA, qB;
    constexpr int HA = G::kOdd ? 0 : 2, HB = G::kOdd ? 1 : 2;
    B4::template front<(1 << NBITS) - 1>(u, p, r, active, A, B, qA, qB);
    const F2 minA = f2_both(qA.mn), invA = f2_both(qA.inv), minB = f2_both(qB.mn), invB = f2_both(qB.inv);
    const F2 magic2 = f2_both(12582912.0f);
    if constexpr (NBITS == 8) {
#pragma unroll
      for (int i = 0; i < G::ITERS; ++i) {
        if (active && G::has(i, ul)) {
          float t0, t1;
          f2_unpack(f2_add(f2_scaled(f2_from_bf16x2(A.w[i]), minA, invA), magic2), t0, t1);
          uint32_t c0 = __float_as_uint(t0) & 0xFFu, c1 = __float_as_uint(t1) & 0xFFu;
          unsigned char* dst = p.codes + 2u * (a0 + ul + UNIT_ * i);
          if (B4::template drop_hi<HA>(i, ul)) dst[0] = (unsigned char)c0;   // the high half is row B's first element
          else *(uint16_t*)dst = (uint16_t)(c0 | (c1 << 8));
          f2_unpack(f2_add(f2_scaled(f2_from_bf16x2(B.w[i]), minB, invB), magic2), t0, t1);
          c0 = __float_as_uint(t0) & 0xFFu;
          c1 = __float_as_uint(t1) & 0xFFu;
          dst = p.codes + 2u * (a1 + ul + UNIT_ * i);
          if (B4::template drop_lo<HB>(i, ul)) dst[1] = (unsigned char)c1;   // the low half is row A's last element
          else *(uint16_t*)dst = (uint16_t)(c0 | (c1 << 8));
        }
      }
      u.sync();
    } else {
      // 2 bits: a word's two codes make a nibble (a foreign half codes as 0), one scratch byte per
      // WORD of the tile; the word the two rows share is written by row B with row A's code merged
      // in (as the 4-bit kernel does with its shared byte).  The warp then packs the scratch of its
      // eight rows, two nibbles to a code byte.
      unsigned char* nibbles = (unsigned char*)tab;
      auto nibble = [&](uint32_t w, bool no_lo, bool no_hi, const QRange& q, F2 min2, F2 inv2) -> uint32_t {
        float v0 = B4::lo(w), v1 = B4::hi(w);
        if (no_lo) v0 = q.mn;
        if (no_hi) v1 = q.mn;
        float t0, t1;
        f2_unpack(f2_add(f2_scaled(f2_pack(v0, v1), min2, inv2), magic2), t0, t1);
        return (__float_as_uint(t0) + (__float_as_uint(t1) << 2)) & 0xFu;  // 0x4B400000 has no bits there
      };
      const uint32_t a_last = nibble(A.w[G::LAST_I], B4::template drop_lo<HA>(G::LAST_I, ul),
                                     B4::template drop_hi<HA>(G::LAST_I, ul), qA, minA, invA);
      const uint32_t shared_lo = __shfl_sync(0xffffffffu, a_last, (threadIdx.x & 31 & ~(UNIT_ - 1)) | G::LAST_UL);
#pragma unroll
      for (int i = 0; i < G::ITERS; ++i) {
        if (active && G::has(i, ul)) {
          if (!G::kOdd || !(i == G::LAST_I && ul == G::LAST_UL))
            nibbles[a0 + ul + UNIT_ * i] = (unsigned char)nibble(A.w[i], B4::template drop_lo<HA>(i, ul),
                                                                 B4::template drop_hi<HA>(i, ul), qA, minA, invA);
          uint32_t b = nibble(B.w[i], B4::template drop_lo<HB>(i, ul), B4::template drop_hi<HB>(i, ul), qB, minB, invB);
          if (G::kOdd && i == 0 && ul == 0) b |= shared_lo & 0x3u;
          nibbles[a1 + ul + UNIT_ * i] = (unsigned char)b;
        }
      }
      u.sync();
      __syncwarp();
      // the warp's eight rows are 4 L words, starting at a multiple of 4 L: four scratch bytes
      // (4-byte aligned) make two code bytes
      const uint32_t w_begin = (grp - (uint32_t)(u.uid & 3)) * (uint32_t)LCT;
      if (active) {
        for (uint32_t b = threadIdx.x & 31u; b < (uint32_t)LCT; b += 32u) {
          const uint32_t w = *(const uint32_t*)(nibbles + w_begin + 4u * b);
          const uint32_t t = (w & 0x000F000Fu) | ((w >> 4) & 0x00F000F0u);   // bytes 0 and 2: the two code bytes
          *(uint16_t*)(p.codes + w_begin / 2u + 2u * b) = (uint16_t)__byte_perm(t, 0u, 0x4420u);
        }
      }
      __syncwarp();
    }
  }
};

template <int DT, int UNIT_, int LCT, int NBITS>
struct PairSoftmaxBwdBits {
  static_assert(NBITS == 2 || NBITS == 8, "4 bits have kernels of their own");
  static constexpr int kMaxRegs = 96;
  static constexpr int kKernel = kSoftmaxBwd;
  static constexpr int UNIT = UNIT_;
  using P = P2<DT>;
  using G = PairGeom<UNIT_, LCT>;
  struct State {};
  static __device__ __forceinline__ void init(State&) {}
  static __device__ __forceinline__ uint32_t rows_per_group(uint32_t) { return 2u; }

  template <int HP>
  static __device__ __forceinline__ void row(Unit<UNIT_>& u, const StagePtrs& p, uint32_t r, bool active) {
    const uint32_t a0 = (r * (uint32_t)LCT) >> 1;
    const int ul = u.ul;
    const float mn = p.meta[2 * r];
    const float s = p.meta[2 * r + 1];
    const F2 mn2 = f2_both(mn), s2 = f2_both(s);
    F2 g[G::ITERS], yh[G::ITERS];
    F2 dot2 = f2_both(0.0f);
#pragma unroll
    for (int i = 0; i < G::ITERS; ++i) {
      float g0 = 0.0f, g1 = 0.0f;
      uint32_t c0 = 0, c1 = 0;
      if (G::has(i, ul)) {
        const uint32_t wd = a0 + ul + UNIT_ * i;           // word of the tile; its elements are 2 wd, 2 wd + 1
        const typename P::Raw w = P::load(p.data, wd);
        g0 = P::lo(w);
        g1 = P::hi(w);
        if (NBITS == 8) {
          const uint32_t b = *(const uint16_t*)(p.codes + 2u * wd);
          c0 = b & 0xFFu;
          c1 = b >> 8;
        } else {
          const uint32_t b = p.codes[wd >> 1] >> (4u * (wd & 1u));   // two words per byte
          c0 = b & 3u;
          c1 = (b >> 2) & 3u;
        }
      }
      if (HP == 1 && i == 0 && ul == 0) g0 = 0.0f;
      if (HP == 0 && i == G::LAST_I && ul == G::LAST_UL) g1 = 0.0f;
      g[i] = f2_pack(g0, g1);
      yh[i] = f2_fma(f2_pack((float)c0, (float)c1), s2, mn2);   // Eq. 9, one rounding each (as dequant)
      dot2 = f2_fma(g[i], yh[i], dot2);
    }
    float d0, d1;
    f2_unpack(dot2, d0, d1);
    const float dot = u.template reduce<kOpSum>(d0 + d1);
    const F2 dotv = f2_both(dot);
#pragma unroll
    for (int i = 0; i < G::ITERS; ++i) {
      if (active && G::has(i, ul)) {
        float o0, o1;
        f2_unpack(f2_mul(yh[i], f2_sub(g[i], dotv)), o0, o1);
        const typename P::Raw w = P::pack(o0, o1);
        const bool drop_lo = HP == 1 && i == 0 && ul == 0;
        const bool drop_hi = HP == 0 && i == G::LAST_I && ul == G::LAST_UL;
        if (drop_lo) P::store_hi(p.data, a0 + ul + UNIT_ * i, w);
        else if (drop_hi) P::store_lo(p.data, a0 + ul + UNIT_ * i, w);
        else P::store(p.data, a0 + ul + UNIT_ * i, w);
      }
    }
  }

  static __device__ __forceinline__ void group(Unit<UNIT_>& u, State&, const StagePtrs& p, float*, uint32_t grp,
                                               bool active, uint32_t) {
    const uint32_t r = active ? 2 * grp : 0;
    if (G::kOdd) {
      row<0>(u, p, r, active);
      u.sync();  // the odd row's first word holds the even row's last result
      row<1>(u, p, r + 1, active);
    } else {
      row<2>(u, p, r, active);
      row<2>(u, p, r + 1, active);
    }
    u.sync();
  }
};

// ---------------------------------------------------------------- the kernel
// RAGGED: the code bytes of a tile need not start on a 16-byte boundary of the code tensor (a
// bulk copy must).  Rows of 1025 elements own 512.5 code bytes each, so only every 32nd row
// starts on such a boundary, and 32 rows of binary32 data are too large a tile to
// double-buffer.  With RAGGED a tile is any even number of rows whose DATA is a multiple of 16
// bytes.  Its codes sit in the stage at the same offset modulo 16 as in global memory
// (code_shift below): the backward loads the 16-byte-aligned span that covers them, the forward
// writes the aligned middle with one bulk store and the up to 15 bytes before and after it
// with plain byte stores of the copy lane.  The kernels that use it access codes bytewise.
struct CodeSpan {
  uint64_t start;    // byte offset of the tile's codes in the code tensor
  uint32_t shift;    // start % 16: where they begin inside the stage's code area
  uint32_t cover;    // bytes of the aligned span covering them (loads)
};
__device__ __forceinline__ CodeSpan code_span(uint64_t tile, uint32_t code_bytes) {
  CodeSpan c;
  c.start = tile * code_bytes;
  c.shift = (uint32_t)c.start & 15u;
  c.cover = (c.shift + code_bytes + 15u) & ~15u;
  return c;
}

template <class WORK, bool RAGGED = false>
__global__ void __maxnreg__(WORK::kMaxRegs) tile_kernel(TileKernelArgs a) {
  extern __shared__ __align__(1024) unsigned char smem[];
  constexpr int KERNEL = WORK::kKernel;
  constexpr int UNIT = WORK::UNIT;
  constexpr bool kFwd = is_fwd(KERNEL);

  uint64_t* full = (uint64_t*)smem;                 // [stages]
  uint64_t* done = (uint64_t*)smem + kMaxStages;    // [stages]
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int n_cwarps = (blockDim.x >> 5) - 1;
  const uint32_t S = a.stages;
  // Tiles go round-robin over the CTAs.  Stage and phase of a tile are carried along the
  // loops (a 64-bit division is a long instruction sequence), and the loops of the frame
  // stay rolled: the four kernels of a training step should fit the instruction cache
  // together.
  const uint64_t my_tiles = a.tiles_per_cta + (blockIdx.x < a.tiles_extra ? 1u : 0u);

  if (threadIdx.x == 0) {
    for (uint32_t s = 0; s < S; ++s) {
      mbar_init(&full[s], 1);
      mbar_init(&done[s], (uint32_t)n_cwarps);
    }
    int* flags = (int*)(smem + kFlagOffset);
    for (int k = 0; k < 16; ++k) flags[k] = 0;
    fence_barrier_init();
    grid_launch_dependents();
  }
  if (threadIdx.x == (uint32_t)n_cwarps * 32u && a.prefetch_tiles != 0) {
    // A CTA that was scheduled while the previous kernel of the stream is still draining
    // uses the time: the inputs of its first tiles are on their way into the L2 when the
    // dependency wait below releases it, which takes the HBM latency out of the pipeline's
    // fill and keeps the read side of the memory busy during the predecessor's last stores.
    const uint32_t pf = my_tiles < a.prefetch_tiles ? (uint32_t)my_tiles : a.prefetch_tiles;
    for (uint32_t i = 0; i < pf; ++i) {
      const uint64_t t = blockIdx.x + (uint64_t)i * gridDim.x;
      bulk_prefetch_l2(a.in + t * a.data_bytes, a.data_bytes);
      if (!kFwd) {
        if (RAGGED) {
          const CodeSpan c = code_span(t, a.code_bytes);
          bulk_prefetch_l2(a.codes + (c.start - c.shift), c.cover);
        } else {
          bulk_prefetch_l2(a.codes + t * a.code_bytes, a.code_bytes);
        }
        bulk_prefetch_l2(a.meta + t * a.meta_bytes, a.meta_bytes);
      }
    }
  }
  __syncthreads();
  // Everything above touched shared memory only or asked for prefetches.  All threads park
  // here (not only the copy lane) so that an early-launched CTA does not spin on its
  // barriers, taking issue slots from the previous kernel's last CTAs.
  grid_dependency_wait();

  if (warp == n_cwarps) {
    // ------------------------------------------------------------ copy warp
    if (lane != 0) return;
    auto issue_load = [&](uint64_t it, uint32_t s) {
      const uint64_t t = blockIdx.x + it * gridDim.x;
      unsigned char* st = smem + kHeaderBytes + (size_t)s * a.stage_bytes;
      uint64_t* bar = &full[s];
      const CodeSpan c = code_span(t, a.code_bytes);
      const uint32_t code_load = RAGGED ? c.cover : a.code_bytes;
      const uint32_t bytes = kFwd ? a.data_bytes : a.data_bytes + code_load + a.meta_bytes;
      mbar_arrive_expect_tx(bar, bytes);
      bulk_load(st, a.in + t * a.data_bytes, a.data_bytes, bar);
      if (!kFwd) {
        bulk_load(st + a.code_off, a.codes + (RAGGED ? c.start - c.shift : c.start), code_load, bar);
        bulk_load(st + a.meta_off, a.meta + t * a.meta_bytes, a.meta_bytes, bar);
      }
    };
    auto prefetch_tile = [&](uint64_t it) {
      const uint64_t t = blockIdx.x + it * gridDim.x;
      bulk_prefetch_l2(a.in + t * a.data_bytes, a.data_bytes);
      if (!kFwd) {
        const CodeSpan c = code_span(t, a.code_bytes);
        bulk_prefetch_l2(a.codes + (RAGGED ? c.start - c.shift : c.start), RAGGED ? c.cover : a.code_bytes);
        bulk_prefetch_l2(a.meta + t * a.meta_bytes, a.meta_bytes);
      }
    };
    const uint32_t pre = my_tiles < S ? (uint32_t)my_tiles : S;
#pragma unroll 1
    for (uint32_t s = 0; s < pre; ++s) issue_load(s, s);
    uint64_t issued = pre;
    uint64_t it = 0;
    uint32_t s = 0, phase = 0;  // stage and phase of tile `it`
    bool ok = true;
#pragma unroll 1
    for (; it < my_tiles; ++it) {
      if (!mbar_wait(&done[s], phase, a.error_word, kErrDrainWait)) { ok = false; break; }
      const uint64_t t = blockIdx.x + it * gridDim.x;
      unsigned char* st = smem + kHeaderBytes + (size_t)s * a.stage_bytes;
      bulk_store(a.out + t * a.data_bytes, st, a.data_bytes);
      if (kFwd) {
        if (RAGGED) {
          const CodeSpan c = code_span(t, a.code_bytes);
          const unsigned char* src = st + a.code_off + c.shift;
          unsigned char* dst = a.codes + c.start;
          const uint32_t head = (16u - c.shift) & 15u;             // bytes before the first boundary
          const uint32_t mid = (a.code_bytes - head) & ~15u;       // whole 16-byte pieces (code_bytes >= 32)
          bulk_store(dst + head, src + head, mid);
#pragma unroll 1
          for (uint32_t k = 0; k < head; ++k) dst[k] = src[k];
#pragma unroll 1
          for (uint32_t k = head + mid; k < a.code_bytes; ++k) dst[k] = src[k];
        } else {
          bulk_store(a.codes + t * a.code_bytes, st + a.code_off, a.code_bytes);
        }
        bulk_store(a.meta + t * a.meta_bytes, st + a.meta_off, a.meta_bytes);
      }
      bulk_commit();
      if (issued < my_tiles) {
        bulk_wait_read<0>();    // the stores of this tile have left shared memory
        issue_load(issued, s);  // tile it + S refills the stage just drained
        if (a.prefetch_ahead != 0 && issued + a.prefetch_ahead < my_tiles) prefetch_tile(issued + a.prefetch_ahead);
        ++issued;
      }
      if (++s == S) { s = 0; phase ^= 1u; }
    }
    bulk_wait_all();
    if (!ok) {
      // wind down: let every load already issued land before shared memory is released
#pragma unroll 1
      for (uint64_t j = it; j < issued; ++j) {
        mbar_wait(&full[s], phase, a.error_word, kErrLoadWait);
        if (++s == S) { s = 0; phase ^= 1u; }
      }
    }
    return;
  }

  // -------------------------------------------------------------- consumer warps
  const int ctid = threadIdx.x;  // consumer warps come first
  Unit<UNIT> u;
  u.ul = ctid % UNIT;
  u.uid = ctid / UNIT;
  u.red = (float*)(smem + kRedOffset) + u.uid * 4;  // [slot(2)][64 floats]; unit k owns floats 4k..4k+3
  u.phase = 0;
  const uint32_t n_units = (uint32_t)(n_cwarps * 32 / UNIT);
  int* abort_flag = (int*)(smem + kFlagOffset) + (UNIT > 32 ? u.uid : 0);
  float* tab = TabFloats<WORK>::value == 16 ? (float*)(smem + kTabOffset) + u.uid * 16
                                            : (float*)(smem + a.tab_off) + u.uid * TabFloats<WORK>::value;
  typename WORK::State state;
  WORK::init(state);

  const uint32_t L = a.row_len;
  const uint32_t n_groups = a.tile_rows / WORK::rows_per_group(L);
  const uint32_t rounds = (n_groups + n_units - 1) / n_units;

  uint32_t s = 0, phase = 0;  // stage and phase of tile `it`
#pragma unroll 1
  for (uint64_t it = 0; it < my_tiles; ++it) {
    bool ok = mbar_wait(&full[s], phase, a.error_word, kErrLoadWait);
    ok = __all_sync(0xffffffffu, ok);
    if (UNIT > 32) {
      if (!ok && lane == 0) *(volatile int*)abort_flag = 1;
      named_bar_sync(1 + u.uid, UNIT);
      ok = *(volatile int*)abort_flag == 0;
    }
    if (!ok) break;
    unsigned char* st = smem + kHeaderBytes + (size_t)s * a.stage_bytes;
    const uint32_t code_shift = RAGGED ? code_span(blockIdx.x + it * gridDim.x, a.code_bytes).shift : 0u;
    StagePtrs sp{st, st + a.code_off + code_shift, (float*)(st + a.meta_off)};
    for (uint32_t rd = 0; rd < rounds; ++rd) {
      uint32_t grp = rd * n_units + u.uid;
      bool active = grp < n_groups;
      if (UNIT < 32 && a.spread_units) {
        // the units of one warp take groups n_groups / (units per warp) apart, which for
        // the odd attention widths puts their words in different shared-memory banks
        constexpr uint32_t upw = 32 / (UNIT < 32 ? UNIT : 32);
        const uint32_t per = n_groups / upw;
        const uint32_t slot = rd * (uint32_t)n_cwarps + (uint32_t)warp;
        grp = (u.uid % upw) * per + slot;
        active = slot < per;
      }
      WORK::group(u, state, sp, tab, grp, active, L);
    }
    fence_proxy_async();  // this thread's shared-memory writes -> visible to the copy engine
    __syncwarp();
    if (lane == 0) mbar_arrive(&done[s]);
    if (++s == S) { s = 0; phase ^= 1u; }
  }
}

// ---------------------------------------------------------------- launching
constexpr uint32_t kMaxSmem = 227 * 1024;

template <class WORK, bool RAGGED = false>
cudaError_t launch_work(const TilePlan& p, const TileKernelArgs& ka, cudaStream_t st) {
  if (RAGGED != (ka.ragged_codes != 0)) return cudaErrorInvalidValue;
  auto kfn = tile_kernel<WORK, RAGGED>;
  // The attributes belong to a device's context: one bit per device and instantiation.  Two
  // threads making the first launch on a device may both set them (the same values).
  static std::atomic<uint64_t> configured{0};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
  if (!(configured.load(std::memory_order_acquire) >> dev & 1ull)) {
    cudaError_t e = cudaFuncSetAttribute(kfn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kMaxSmem);
    if (e != cudaSuccess) return e;
    // Always the largest shared-memory carve-out: kernels of different kinds then leave the
    // SMs in the same configuration, and consecutive launches need no reconfiguration.
    e = cudaFuncSetAttribute(kfn, cudaFuncAttributePreferredSharedMemoryCarveout, (int)cudaSharedmemCarveoutMaxShared);
    if (e != cudaSuccess) return e;
    configured.fetch_or(1ull << dev, std::memory_order_release);
  }
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(p.grid);
  cfg.blockDim = dim3((p.warps + 1) * 32);
  cfg.dynamicSmemBytes = p.smem_bytes;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = p.overlap_launch ? 1 : 0;
  return cudaLaunchKernelEx(&cfg, kfn, ka);
}

// The general policy, by unit size and register bound.
template <int KERNEL, int DT, int VMODE, int UNIT>
cudaError_t launch_generic_iters(const TilePlan& p, const TileKernelArgs& ka, cudaStream_t st) {
  constexpr int kMax = (DT == kBF16 && VMODE == kVec16) ? 8 : 16;  // elements per lane stay <= 64
  switch (p.iters) {
    case 1: return launch_work<GenericWork<KERNEL, DT, VMODE, UNIT, 1>>(p, ka, st);
    case 2: return launch_work<GenericWork<KERNEL, DT, VMODE, UNIT, 2>>(p, ka, st);
    case 4: return launch_work<GenericWork<KERNEL, DT, VMODE, UNIT, 4>>(p, ka, st);
    case 8: return launch_work<GenericWork<KERNEL, DT, VMODE, UNIT, 8>>(p, ka, st);
    case 16:
      if (kMax >= 16) return launch_work<GenericWork<KERNEL, DT, VMODE, UNIT, kMax>>(p, ka, st);
  }
  return cudaErrorInvalidValue;
}

template <int KERNEL, int DT>
cudaError_t launch_generic(const TilePlan& p, const TileKernelArgs& ka, cudaStream_t st) {
  if (p.vec_elems == 2) {
    switch (p.unit_lanes) {
      case 8: return launch_generic_iters<KERNEL, DT, kPair, 8>(p, ka, st);
      case 32: return launch_generic_iters<KERNEL, DT, kPair, 32>(p, ka, st);
    }
  } else if constexpr (KERNEL == kSoftmaxFwd || KERNEL == kSoftmaxBwd) {
    if (p.unit_lanes == 128) return launch_generic_iters<KERNEL, DT, kVec16, 128>(p, ka, st);
  }
  return cudaErrorInvalidValue;
}

template <template <int, int, int> class WORK, int DT, int UNIT>
cudaError_t launch_softmax_nv(const TilePlan& p, const TileKernelArgs& ka, cudaStream_t st) {
  switch (p.iters) {
    case 1: return launch_work<WORK<DT, UNIT, 1>>(p, ka, st);
    case 2: return launch_work<WORK<DT, UNIT, 2>>(p, ka, st);
    case 4: return launch_work<WORK<DT, UNIT, 4>>(p, ka, st);
    case 8: return launch_work<WORK<DT, UNIT, 8>>(p, ka, st);
    case 16:
      if (DT == kF32) return launch_work<WORK<DT, UNIT, DT == kF32 ? 16 : 8>>(p, ka, st);
  }
  return cudaErrorInvalidValue;
}

// Multi-warp units take the long rows: 4 or 8 vectors per lane (16 for binary32 at 8192).
template <template <int, int, int> class WORK, int DT, int UNIT>
cudaError_t launch_softmax_wide(const TilePlan& p, const TileKernelArgs& ka, cudaStream_t st) {
  switch (p.iters) {
    case 4: return launch_work<WORK<DT, UNIT, 4>>(p, ka, st);
    case 8: return launch_work<WORK<DT, UNIT, 8>>(p, ka, st);
    case 16:
      if (DT == kF32 && UNIT == 128) return launch_work<WORK<DT, UNIT, DT == kF32 ? 16 : 8>>(p, ka, st);
  }
  return cudaErrorInvalidValue;
}

// Units of 2 or 4 lanes take the very short rows: 2 or 4 vectors per lane.
template <template <int, int, int> class WORK, int DT, int UNIT>
cudaError_t launch_softmax_narrow(const TilePlan& p, const TileKernelArgs& ka, cudaStream_t st) {
  switch (p.iters) {
    case 2: return launch_work<WORK<DT, UNIT, 2>>(p, ka, st);
    case 4: return launch_work<WORK<DT, UNIT, 4>>(p, ka, st);
  }
  return cudaErrorInvalidValue;
}

template <template <int, int, int> class WORK, int DT>
cudaError_t launch_softmax_stream(const TilePlan& p, const TileKernelArgs& ka, cudaStream_t st) {
  switch (p.unit_lanes) {
    case 2: return launch_softmax_narrow<WORK, DT, 2>(p, ka, st);
    case 4: return launch_softmax_narrow<WORK, DT, 4>(p, ka, st);
    case 8: return launch_softmax_nv<WORK, DT, 8>(p, ka, st);
    case 16: return launch_softmax_nv<WORK, DT, 16>(p, ka, st);
    case 32: return launch_softmax_nv<WORK, DT, 32>(p, ka, st);
    case 64: return launch_softmax_wide<WORK, DT, 64>(p, ka, st);
    case 128: return launch_softmax_wide<WORK, DT, 128>(p, ka, st);
  }
  return cudaErrorInvalidValue;
}

template <template <int, int, int> class WORK, int DT, int UNIT>
cudaError_t launch_gelu_nvl(const TilePlan& p, const TileKernelArgs& ka, cudaStream_t st) {
  if (UNIT >= 64) {  // fixed vector counts exist for the multi-warp units only
    constexpr int U = UNIT >= 64 ? UNIT : 64;
    switch (p.iters) {
      case 3: return launch_work<WORK<DT, U, 3>>(p, ka, st);
      case 4: return launch_work<WORK<DT, U, 4>>(p, ka, st);
      case 5: return launch_work<WORK<DT, U, 5>>(p, ka, st);
      case 6: return launch_work<WORK<DT, U, 6>>(p, ka, st);
      case 8: return launch_work<WORK<DT, U, 8>>(p, ka, st);
      case 10: return launch_work<WORK<DT, U, 10>>(p, ka, st);
    }
  }
  return launch_work<WORK<DT, UNIT, 0>>(p, ka, st);
}

template <template <int, int, int> class WORK, int DT>
cudaError_t launch_gelu_stream(const TilePlan& p, const TileKernelArgs& ka, cudaStream_t st) {
  switch (p.unit_lanes) {
    case 8: return launch_gelu_nvl<WORK, DT, 8>(p, ka, st);
    case 16: return launch_gelu_nvl<WORK, DT, 16>(p, ka, st);
    case 32: return launch_gelu_nvl<WORK, DT, 32>(p, ka, st);
    case 64: return launch_gelu_nvl<WORK, DT, 64>(p, ka, st);
    case 128: return launch_gelu_nvl<WORK, DT, 128>(p, ka, st);
  }
  return cudaErrorInvalidValue;
}

template <template <int, int, int> class WORK, int DT>
cudaError_t launch_pair_fixed(const TilePlan& p, const TileKernelArgs& ka, cudaStream_t st) {
  if (p.unit_lanes != 8) return cudaErrorInvalidValue;
  switch (ka.row_len) {
    case 197: return launch_work<WORK<DT, 8, 197>>(p, ka, st);
    case 257: return launch_work<WORK<DT, 8, 257>>(p, ka, st);
  }
  return cudaErrorInvalidValue;
}

// The other fixed widths (instantiated in a translation unit of their own).
template <template <int, int, int> class WORK, int DT>
cudaError_t launch_pair_widths(const TilePlan& p, const TileKernelArgs& ka, cudaStream_t st) {
  if (p.unit_lanes == 32) {  // the long widths: a warp per row pair
    switch (ka.row_len) {
      case 577:
        return ka.ragged_codes ? launch_work<WORK<DT, 32, 577>, true>(p, ka, st) : launch_work<WORK<DT, 32, 577>>(p, ka, st);
      case 1025:
        return ka.ragged_codes ? launch_work<WORK<DT, 32, 1025>, true>(p, ka, st) : launch_work<WORK<DT, 32, 1025>>(p, ka, st);
    }
    return cudaErrorInvalidValue;
  }
  if (p.unit_lanes == 4) {  // the short widths, forward: four lanes per row
    if constexpr (WORK<DT, 4, 49>::kKernel == kSoftmaxFwd) {
      switch (ka.row_len) {
        case 49: return launch_work<WORK<DT, 4, 49>>(p, ka, st);
        case 50: return launch_work<WORK<DT, 4, 50>>(p, ka, st);
      }
    }
    return cudaErrorInvalidValue;
  }
  if (p.unit_lanes != 8) return cudaErrorInvalidValue;
  switch (ka.row_len) {
    case 49: return launch_work<WORK<DT, 8, 49>>(p, ka, st);
    case 50: return launch_work<WORK<DT, 8, 50>>(p, ka, st);
    case 145: return launch_work<WORK<DT, 8, 145>>(p, ka, st);
    case 196: return launch_work<WORK<DT, 8, 196>>(p, ka, st);
    case 198: return launch_work<WORK<DT, 8, 198>>(p, ka, st);
  }
  return cudaErrorInvalidValue;
}
template <int KERNEL>
cudaError_t launch_tile_pair_widths_kernel(int dt, const TilePlan& p, const TileKernelArgs& ka, cudaStream_t st) {
  if constexpr (KERNEL == kSoftmaxFwd)
    return dt == kF32 ? launch_pair_widths<PairSoftmaxFwd, kF32>(p, ka, st) : launch_pair_widths<PairSoftmaxFwd, kBF16>(p, ka, st);
  else
    return dt == kF32 ? launch_pair_widths<PairSoftmaxBwd, kF32>(p, ka, st) : launch_pair_widths<PairSoftmaxBwd, kBF16>(p, ka, st);
}

template <template <int, int> class WORK, int DT>
cudaError_t launch_any(const TilePlan& p, const TileKernelArgs& ka, cudaStream_t st) {
  switch (p.unit_lanes) {
    case 1: return launch_work<WORK<DT, 1>>(p, ka, st);
    case 2: return launch_work<WORK<DT, 2>>(p, ka, st);
    case 4: return launch_work<WORK<DT, 4>>(p, ka, st);
    case 8: return launch_work<WORK<DT, 8>>(p, ka, st);
    case 16: return launch_work<WORK<DT, 16>>(p, ka, st);
    case 32: return launch_work<WORK<DT, 32>>(p, ka, st);
    case 64: return launch_work<WORK<DT, 64>>(p, ka, st);
    case 128: return launch_work<WORK<DT, 128>>(p, ka, st);
  }
  return cudaErrorInvalidValue;
}

template <int KERNEL, int DT>
cudaError_t launch_variant(const TilePlan& p, const TileKernelArgs& ka, cudaStream_t st) {
  if (p.variant == kVariantAny) {
    if constexpr (KERNEL == kSoftmaxFwd) return launch_any<AnySoftmaxFwd, DT>(p, ka, st);
    if constexpr (KERNEL == kSoftmaxBwd) return launch_any<AnySoftmaxBwd, DT>(p, ka, st);
    return cudaErrorInvalidValue;
  }
  if (p.variant == kVariantStream) {
    if constexpr (KERNEL == kGeluFwd) return launch_gelu_stream<StreamGeluFwd, DT>(p, ka, st);
    if constexpr (KERNEL == kGeluBwd) return launch_gelu_stream<StreamGeluBwd, DT>(p, ka, st);
    if constexpr (KERNEL == kSoftmaxFwd) return launch_softmax_stream<StreamSoftmaxFwd, DT>(p, ka, st);
    if constexpr (KERNEL == kSoftmaxBwd) return launch_softmax_stream<StreamSoftmaxBwd, DT>(p, ka, st);
    if constexpr (KERNEL == kSiluFwd) return launch_gelu_stream<StreamSiluFwd, DT>(p, ka, st);
    if constexpr (KERNEL == kSiluBwd) return launch_gelu_stream<StreamSiluBwd, DT>(p, ka, st);
  }
  if constexpr (KERNEL == kSiluFwd || KERNEL == kSiluBwd) return cudaErrorInvalidValue;  // streamed form only
  if (p.variant == kVariantPairFixed) {
    if constexpr (KERNEL == kSoftmaxFwd) return launch_pair_fixed<PairSoftmaxFwd, DT>(p, ka, st);
    if constexpr (KERNEL == kSoftmaxBwd) return launch_pair_fixed<PairSoftmaxBwd, DT>(p, ka, st);
    return cudaErrorInvalidValue;
  }
  return launch_generic<KERNEL, DT>(p, ka, st);
}

// The 2- and 8-bit GELU kernels (their own translation unit instantiates this).
template <template <int, int, int> class WORK, int DT, int NBITS>
cudaError_t launch_any_bits(const TilePlan& p, const TileKernelArgs& ka, cudaStream_t st) {
  switch (p.unit_lanes) {
    case 2: return launch_work<WORK<DT, 2, NBITS>>(p, ka, st);
    case 4: return launch_work<WORK<DT, 4, NBITS>>(p, ka, st);
    case 8: return launch_work<WORK<DT, 8, NBITS>>(p, ka, st);
    case 16: return launch_work<WORK<DT, 16, NBITS>>(p, ka, st);
    case 32: return launch_work<WORK<DT, 32, NBITS>>(p, ka, st);
  }
  return cudaErrorInvalidValue;
}

template <int KERNEL, int DT, int NBITS>
cudaError_t launch_bits_unit(const TilePlan& p, const TileKernelArgs& ka, cudaStream_t st) {
  if constexpr (KERNEL == kSoftmaxFwd) {
    if (p.variant == kVariantPairFixed) {
      if (ka.row_len == 197) return launch_work<PairSoftmaxFwdBits<DT, 8, 197, NBITS>>(p, ka, st);
      if (ka.row_len == 257) return launch_work<PairSoftmaxFwdBits<DT, 8, 257, NBITS>>(p, ka, st);
      return cudaErrorInvalidValue;
    }
    return launch_any_bits<AnySoftmaxFwdBits, DT, NBITS>(p, ka, st);
  } else if constexpr (KERNEL == kSoftmaxBwd) {
    if (p.variant == kVariantPairFixed) {
      if (ka.row_len == 197) return launch_work<PairSoftmaxBwdBits<DT, 8, 197, NBITS>>(p, ka, st);
      if (ka.row_len == 257) return launch_work<PairSoftmaxBwdBits<DT, 8, 257, NBITS>>(p, ka, st);
      return cudaErrorInvalidValue;
    }
    return launch_any_bits<AnySoftmaxBwdBits, DT, NBITS>(p, ka, st);
  } else if constexpr (KERNEL == kGeluFwd) {
    if (p.unit_lanes == 64) return launch_work<StreamActFwdBits<DT, 64, kActGelu, NBITS>>(p, ka, st);
    if (p.unit_lanes == 128) return launch_work<StreamActFwdBits<DT, 128, kActGelu, NBITS>>(p, ka, st);
  } else {
    if (p.unit_lanes == 64) return launch_work<StreamActBwdBits<DT, 64, kActGelu, NBITS>>(p, ka, st);
    if (p.unit_lanes == 128) return launch_work<StreamActBwdBits<DT, 128, kActGelu, NBITS>>(p, ka, st);
  }
  return cudaErrorInvalidValue;
}
template <int KERNEL>
cudaError_t launch_tile_bits_kernel(int dt, const TilePlan& p, const TileKernelArgs& ka, cudaStream_t st) {
  if (p.bits == 2)
    return dt == kF32 ? launch_bits_unit<KERNEL, kF32, 2>(p, ka, st) : launch_bits_unit<KERNEL, kBF16, 2>(p, ka, st);
  if (p.bits == 8)
    return dt == kF32 ? launch_bits_unit<KERNEL, kF32, 8>(p, ka, st) : launch_bits_unit<KERNEL, kBF16, 8>(p, ka, st);
  return cudaErrorInvalidValue;
}

// One translation unit per entry point instantiates this.
template <int KERNEL>
cudaError_t launch_tile_kernel(int dt, const TilePlan& p, const TileKernelArgs& ka, cudaStream_t st) {
  return dt == kF32 ? launch_variant<KERNEL, kF32>(p, ka, st) : launch_variant<KERNEL, kBF16>(p, ka, st);
}

}  // namespace
}  // namespace s2a
