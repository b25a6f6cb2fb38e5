// Device-side building blocks shared by the S2A kernels: I/O type traits, the Eq. 8
// quantiser in pinned binary32 operations, Eq. 10 / Eq. 12 arithmetic, reductions.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace s2a {

constexpr int kF32 = 0;
constexpr int kBF16 = 1;

constexpr float kSlope = 1.702f;   // Eq. 10 / Eq. 12: sigmoid(1.702 x)
constexpr float kSineAmp = 0.22f;  // Eq. 12: 0.22 sin(1.5 x)
constexpr float kSineFreq = 1.5f;
constexpr float kClip = 2.0f;      // Section 3.2: GELU input clipped into [-2, 2]
constexpr float kLevels = 15.0f;   // 2^N - 1 with N = 4 (Eq. 8)

// Bits of the per-device error word (see s2a_device_error).
constexpr unsigned kErrLoadWait = 1u;   // a consumer gave up waiting for a tile to arrive
constexpr unsigned kErrDrainWait = 2u;  // the producer gave up waiting for the consumers
constexpr unsigned kErrSelfTest = 4u;   // set by s2a_selftest_wait_expiry only: its wait is meant to run out

// ---------------------------------------------------------------- I/O element types
template <int DT> struct Io;
template <> struct Io<kF32> {
  using T = float;
  static constexpr int kBytes = 4;
  static __device__ __forceinline__ float widen(float v) { return v; }
  static __device__ __forceinline__ float narrow(float v) { return v; }
};
template <> struct Io<kBF16> {
  using T = __nv_bfloat16;
  static constexpr int kBytes = 2;
  static __device__ __forceinline__ float widen(__nv_bfloat16 v) { return __bfloat162float(v); }
  static __device__ __forceinline__ __nv_bfloat16 narrow(float v) { return __float2bfloat16_rn(v); }
};

// ---------------------------------------------------------------- Eq. 8 quantiser
// Specified as correctly rounded binary32 steps; the intrinsics keep the compiler from
// contracting the subtract and the multiply into one fused operation.
struct QRange {
  float mn;   // min of the row
  float inv;  // 15 / (max - min), 0 for a constant row
  float s;    // (max - min) / 15, 0 for a constant row
};

__device__ __forceinline__ QRange make_qrange(float mn, float mx, float levels = kLevels) {
  QRange q;
  q.mn = mn;
  float d = __fsub_rn(mx, mn);
  if (d == 0.0f) {
    q.inv = 0.0f;
    q.s = 0.0f;
  } else {
    q.inv = __fdiv_rn(levels, d);
    q.s = __fdiv_rn(d, levels);
  }
  return q;
}

// For v inside [min, max] the scaled value lies in [0, 15 + 2^-20], so adding
// 1.5 * 2^23 rounds it half-to-even into the low mantissa bits without a clamp.
__device__ __forceinline__ uint32_t quant_code(float v, const QRange& q, uint32_t mask = 0xFu) {
  float t = __fmul_rn(__fsub_rn(v, q.mn), q.inv);
  return __float_as_uint(__fadd_rn(t, 12582912.0f)) & mask;
}

// Eq. 9 in binary32: one rounding of the exact code * s + min.
__device__ __forceinline__ float dequant(uint32_t code, float mn, float s) {
  return __fmaf_rn((float)code, s, mn);
}

// ---------------------------------------------------------------- Eq. 10 and Eq. 12
// The two input-stash activations.  GELU is the paper's x * sigmoid(1.702 x) with the
// sine-fitted derivative of Eq. 12 and the clip [-2, 2].  SiLU (x * sigmoid(x)) is named by
// the paper without constants: it is given the clip 2 * 1.702 (the same range of the
// sigmoid's argument) and its exact derivative.
enum { kActGelu = 0, kActSilu = 1 };
template <int ACT> struct Act;
template <> struct Act<kActGelu> {
  static constexpr float kSlopeOf = kSlope;
  static constexpr float kClipOf = kClip;
};
template <> struct Act<kActSilu> {
  static constexpr float kSlopeOf = 1.0f;
  static constexpr float kClipOf = 2.0f * 1.702f;
};

// y = x * sigmoid(a x), evaluated through t = exp(-|a x|) so that neither tail
// overflows: sigmoid(z) = 1 / (1 + t) for z >= 0 and t / (1 + t) for z < 0.  The
// product a x is carried as hi + lo so that its rounding does not scale the error
// of exp with |x|.
template <int ACT>
__device__ __forceinline__ float act_value(float x) {
  constexpr float a = Act<ACT>::kSlopeOf;
  float z = __fmul_rn(a, x);
  float zlo = __fmaf_rn(a, x, -z);
  float t = expf(-fabsf(z)) * (1.0f - (z >= 0.0f ? zlo : -zlo));
  // a / b with b = 1 + t in [1, 2]: the hardware reciprocal (1 ulp) and one correction step
  // on the remainder, which leaves about an ulp -- no special cases can arise for such b
  const float a_num = z >= 0.0f ? x : x * t, b_den = 1.0f + t;
  float r;
  asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(b_den));
  const float q = a_num * r;
  return __fmaf_rn(__fmaf_rn(-b_den, q, a_num), r, q);
}
__device__ __forceinline__ float gelu_value(float x) { return act_value<kActGelu>(x); }

// Fast forms for bfloat16 outputs (the result is rounded to 8 bits): one special-function
// exponential and one reciprocal.
__device__ __forceinline__ float ex2_approx(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ float rcp_approx(float x) {
  float y;
  asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// y = x / (1 + 2^k), k = -a log2(e) x.  Both forms below are for bfloat16 outputs.
//
// The short form is exact enough while 2^k is finite and 1 / 2^k is a normal number, i.e.
// for k <= 126 (x >= kFastFloor): beyond that ex2.approx returns +inf (or rcp.approx.ftz
// flushes a subnormal reciprocal) and y would come out as -0 although its true magnitude,
// |x| 2^-k, is still a normal bfloat16 number down to k = 126 + log2|x|.  Callers use it
// only on rows whose minimum is at or above kFastFloor.
template <int ACT>
struct ActFast {
  static constexpr float kC = -Act<ACT>::kSlopeOf * 1.4426950408889634f;
  static constexpr float kFastFloor = -125.0f / (Act<ACT>::kSlopeOf * 1.4426950408889634f);
  static __device__ __forceinline__ float eval(float x) { return x * rcp_approx(1.0f + ex2_approx(kC * x)); }
};

// The general form carries the denominator scaled by 2^-8: 2^-8 + 2^(k-8) stays finite, and
// its reciprocal normal, up to k = 134; from there on |y| = |x| 2^-k is below 2^-126 (k = 134
// is reached at |x| = 92.9 / a), so only results below the normal range flush to zero.
template <int DT, int ACT = kActGelu>
__device__ __forceinline__ float gelu_eval(float x) {
  if (DT == kF32) return act_value<ACT>(x);
  const float w = 0.00390625f + ex2_approx(__fmaf_rn(ActFast<ACT>::kC, x, -8.0f));
  return (x * rcp_approx(w)) * 0.00390625f;
}

// The derivative used by the backward pass at a dequantised x_hat = code * s + min, in
// binary64: Eq. 12 for GELU, the exact derivative for SiLU.
template <int ACT>
__device__ __forceinline__ double act_derivative(uint32_t code, float mn, float s) {
  double xh = (double)code * (double)s + (double)mn;
  if (ACT == kActGelu) {
    double sig = 1.0 / (1.0 + exp(-(double)kSlope * xh));
    return sig + (double)kSineAmp * sin((double)kSineFreq * xh);
  }
  double sig = 1.0 / (1.0 + exp(-xh));
  return sig * (1.0 + xh * (1.0 - sig));
}
__device__ __forceinline__ double gelu_sine_derivative(uint32_t code, float mn, float s) {
  return act_derivative<kActGelu>(code, mn, s);
}

// ---------------------------------------------------------------- packed binary32 pairs
// sm_100 executes add / sub / mul / fma on TWO binary32 values held in a 64-bit register
// pair with one instruction, each half correctly rounded exactly like the scalar operation
// (so the pinned operation sequence of Eq. 8 keeps its results bit for bit).  The kernels
// are bound by instruction issue as much as by memory, and this halves the issue slots of
// their floating-point arithmetic.
struct F2 {
  uint64_t v;
};
__device__ __forceinline__ F2 f2_pack(float lo, float hi) {
  F2 r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r.v) : "f"(lo), "f"(hi));
  return r;
}
__device__ __forceinline__ F2 f2_both(float x) { return f2_pack(x, x); }
__device__ __forceinline__ void f2_unpack(F2 a, float& lo, float& hi) {
  asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(a.v));
}
__device__ __forceinline__ F2 f2_fma(F2 a, F2 b, F2 c) {
  F2 d;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d.v) : "l"(a.v), "l"(b.v), "l"(c.v));
  return d;
}
__device__ __forceinline__ F2 f2_add(F2 a, F2 b) {
  F2 d;
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d.v) : "l"(a.v), "l"(b.v));
  return d;
}
__device__ __forceinline__ F2 f2_sub(F2 a, F2 b) {
  F2 d;
  asm("sub.rn.f32x2 %0, %1, %2;" : "=l"(d.v) : "l"(a.v), "l"(b.v));
  return d;
}
__device__ __forceinline__ F2 f2_mul(F2 a, F2 b) {
  F2 d;
  asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(d.v) : "l"(a.v), "l"(b.v));
  return d;
}
// The two halves of a packed bfloat16 pair, widened (exact).
__device__ __forceinline__ F2 f2_from_bf16x2(uint32_t w) {
  return f2_pack(__uint_as_float(w << 16), __uint_as_float(w & 0xffff0000u));
}
// Rounds both halves to bfloat16 (nearest even): low half in the low 16 bits.
__device__ __forceinline__ uint32_t f2_to_bf16x2(F2 a) {
  float lo, hi;
  f2_unpack(a, lo, hi);
  __nv_bfloat162 b = __floats2bfloat162_rn(lo, hi);
  return *(uint32_t*)&b;
}
// Eq. 8 on a pair: (code of lo) + 16 * (code of hi) + a constant the caller removes or
// ignores above bit 7 -- the rounded scaled values sit in the low mantissa bits of
// t + 1.5 * 2^23 (see quant_code).  min2 / inv2 hold the row's min and 15 / (max - min) twice.
//
// The product is formed by an fma with +0 (the same value as the multiply: the scaled values
// are never -0).  A packed multiply followed directly by a packed add is contracted by the
// assembler into ONE fused operation, explicit rounding modifiers notwithstanding (measured:
// 7e-4 of random pairs then differ), and a single rounding breaks the ties that Eq. 8's
// pinned sequence resolves with two: a product that rounds to exactly k + 1/2 must go to the
// even code.  An fma result is not contracted further.
__device__ __forceinline__ F2 f2_scaled(F2 v, F2 min2, F2 inv2) {
  return f2_fma(f2_sub(v, min2), inv2, f2_both(0.0f));
}
__device__ __forceinline__ uint32_t f2_code_byte(F2 v, F2 min2, F2 inv2) {
  const F2 t = f2_add(f2_scaled(v, min2, inv2), f2_both(12582912.0f));
  float lo, hi;
  f2_unpack(t, lo, hi);
  return __float_as_uint(lo) + (__float_as_uint(hi) << 4);  // bits 0..7: the two codes (0x4B400000 has none there)
}

// Packed pair forms of the bfloat16 activation (see ActFast / gelu_eval for the two ranges).
template <int ACT>
__device__ __forceinline__ F2 f2_act_fast(F2 x) {
  float k0, k1, d0, d1;
  f2_unpack(f2_mul(x, f2_both(ActFast<ACT>::kC)), k0, k1);
  f2_unpack(f2_add(f2_pack(ex2_approx(k0), ex2_approx(k1)), f2_both(1.0f)), d0, d1);
  return f2_mul(x, f2_pack(rcp_approx(d0), rcp_approx(d1)));
}
// Four elements per call, two elements per reciprocal: 1 / (d0 d1) and two multiplications give
// 1 / d0 and 1 / d1.  The forward kernel's row work is bound by instruction issue first and by the
// special-function unit (a quarter of the other pipes' rate) second; measured on the ViT-B/16
// GELU launch at sustained clocks: a reciprocal per element (8 special-function operations per four
// elements) 31.3 us, one per four elements (5 operations, seven multiplications) 30.6 us, one per
// pair (6 operations, four multiplications) 30.3 us.  Each d_i = 1 + 2^k_i: callers use this on
// rows whose minimum is at or above kQuadFloor (k <= 30), so that a product stays far from overflow.
template <int ACT>
struct ActQuad {
  static constexpr float kQuadFloor = -30.0f / (Act<ACT>::kSlopeOf * 1.4426950408889634f);
  static __device__ __forceinline__ void eval(F2 xa, F2 xb, F2& ya, F2& yb) {
    const F2 c2 = f2_both(ActFast<ACT>::kC), one2 = f2_both(1.0f);
    float k0, k1, k2, k3, d0, d1, d2, d3;
    f2_unpack(f2_mul(xa, c2), k0, k1);
    f2_unpack(f2_mul(xb, c2), k2, k3);
    f2_unpack(f2_add(f2_pack(ex2_approx(k0), ex2_approx(k1)), one2), d0, d1);
    f2_unpack(f2_add(f2_pack(ex2_approx(k2), ex2_approx(k3)), one2), d2, d3);
    const float ra = rcp_approx(d0 * d1), rb = rcp_approx(d2 * d3);
    ya = f2_mul(xa, f2_mul(f2_pack(d1, d0), f2_both(ra)));   // x0 / d0, x1 / d1
    yb = f2_mul(xb, f2_mul(f2_pack(d3, d2), f2_both(rb)));
  }
};

template <int ACT>
__device__ __forceinline__ F2 f2_act_general(F2 x) {
  float k0, k1, d0, d1;
  f2_unpack(f2_fma(x, f2_both(ActFast<ACT>::kC), f2_both(-8.0f)), k0, k1);
  f2_unpack(f2_add(f2_pack(ex2_approx(k0), ex2_approx(k1)), f2_both(0.00390625f)), d0, d1);
  return f2_mul(f2_mul(x, f2_pack(rcp_approx(d0), rcp_approx(d1))), f2_both(0.00390625f));
}
__device__ __forceinline__ F2 f2_clip(F2 x, float c) {
  float a, b;
  f2_unpack(x, a, b);
  return f2_pack(fminf(fmaxf(a, -c), c), fminf(fmaxf(b, -c), c));
}

// ---------------------------------------------------------------- warp reductions
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}
__device__ __forceinline__ float warp_min(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fminf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

}  // namespace s2a
