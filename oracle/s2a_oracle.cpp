// S2A 4-bit activation stash -- CPU ORACLE.  TEST INFRASTRUCTURE, NOT THE PRODUCT.
//
// A plain, slow, scalar restatement of the paper's Section 3.2 ("Non-Parametric
// Layers") for GELU and softmax: the forward evaluates the nonlinearity and keeps a
// 4-bit code of what backward needs; the backward dequantises the code and forms the
// input gradient.  It exists only so that tests, the smoke check and the benchmark's
// CPU-baseline leg can compare the CUDA library against something written directly
// from the paper.  It shares no source, header, table or helper with the CUDA path
// and must never be reached from it.
//
// Arithmetic: every real-valued step is evaluated in binary64 and rounded ONCE to the
// I/O type (binary32 or bfloat16, round-to-nearest-even).  The quantiser is the one
// exception: it is specified as a sequence of correctly rounded binary32 operations
// (see quantize_row) so that an independent implementation can reproduce its codes
// bit for bit.  Compile with -O2 -ffp-contract=off and never with -ffast-math.
//
// Parity status: every function below is pinned by tests that do not call it to
// produce their expected values (closed forms, exact rational arithmetic, library
// routines, finite differences, hand-worked rows).  The accuracy figures the paper
// reports for trained networks are "parity unpinned": they need datasets and
// pretrained weights that are not available.

#include <algorithm>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <thread>
#include <vector>

namespace {

enum { DT_F32 = 0, DT_BF16 = 1 };

// Constants as the binary32 numbers nearest to the decimals printed in Eq. 10 and
// Eq. 12 (1.702, 0.22, 1.5), widened exactly to binary64.
const double kA = (double)1.702f;   // sigmoid slope, Eq. 10 / Eq. 12
const double kB = (double)0.22f;    // sine amplitude, Eq. 12
const double kW = (double)1.5f;     // sine frequency, Eq. 12
const int kBits = 4;                // N in Eq. 8 (Section 4.1: 4-bit)
const int kLevels = (1 << kBits) - 1;  // 2^N - 1 = 15

// ---------------------------------------------------------------- number formats

float bf16_bits_to_float(uint16_t b) {
  uint32_t u = (uint32_t)b << 16;
  float f;
  std::memcpy(&f, &u, 4);
  return f;
}

// binary64 -> bfloat16, round-to-nearest-even, in ONE rounding (no detour through
// binary32, which would round twice).  bfloat16: 8 significant bits, binary32's
// exponent range, gradual underflow below 2^-126.
uint16_t round_to_bf16_bits(double d) {
  if (std::isnan(d)) return 0x7FC0;
  uint16_t sign = std::signbit(d) ? 0x8000 : 0;
  double a = std::fabs(d);
  if (a == 0.0) return sign;
  if (std::isinf(a)) return sign | 0x7F80;
  int e = std::ilogb(a);
  if (e < -126) e = -126;                    // subnormal spacing
  double quantum = std::ldexp(1.0, e - 7);   // distance between neighbours
  double r = std::nearbyint(a / quantum);    // default rounding mode: ties-to-even
  double v = r * quantum;                    // exact
  const double max_bf16 = std::ldexp(255.0, 127 - 7);  // (2 - 2^-7) * 2^127
  if (v > max_bf16) return sign | 0x7F80;
  float f = (float)v;                        // exact: v is a bfloat16 value
  uint32_t u;
  std::memcpy(&u, &f, 4);
  return sign | (uint16_t)(u >> 16);
}

double load_elem(const void* p, size_t i, int dt) {
  if (dt == DT_F32) return (double)((const float*)p)[i];
  return (double)bf16_bits_to_float(((const uint16_t*)p)[i]);
}

// Round a binary64 result once to the I/O type, store it, and return the stored
// value widened back (the value "as written").
float store_elem(void* p, size_t i, int dt, double v) {
  if (dt == DT_F32) {
    float f = (float)v;  // correctly rounded (round-to-nearest-even)
    ((float*)p)[i] = f;
    return f;
  }
  uint16_t b = round_to_bf16_bits(v);
  ((uint16_t*)p)[i] = b;
  return bf16_bits_to_float(b);
}

// ---------------------------------------------------------------- the nonlinearities

double sigmoid(double z) { return 1.0 / (1.0 + std::exp(-z)); }

// Eq. 10: y = x * sigmoid(1.702 x).
double gelu(double x) { return x * sigmoid(kA * x); }

// Eq. 11: the exact derivative of Eq. 10 (never executed on the stash path; kept so
// that tests can check Eq. 10 against finite differences and Eq. 12 against it).
double gelu_grad_exact(double x) {
  double z = kA * x;
  double s = sigmoid(z);
  return s + z * std::exp(-z) * s * s;
}

// Eq. 12: sigmoid(1.702 x) + 0.22 sin(1.5 x), the sine-fitted derivative.
double gelu_grad_sine(double x) { return sigmoid(kA * x) + kB * std::sin(kW * x); }

// Eq. 7, forward: y_i = exp(x_i) / sum_j exp(x_j).  The row maximum is subtracted
// first, which leaves the quotient unchanged and keeps exp in range.
void softmax_row(const double* x, double* y, size_t n) {
  double m = x[0];
  for (size_t j = 1; j < n; ++j) m = std::max(m, x[j]);
  double Z = 0.0;
  for (size_t j = 0; j < n; ++j) {
    y[j] = std::exp(x[j] - m);
    Z += y[j];
  }
  for (size_t j = 0; j < n; ++j) y[j] /= Z;
}

// Eq. 7, Jacobian applied to g:  grad_in_i = sum_j g_j dy_j/dx_i with
// dy_j/dx_i = y_j (delta_ij - y_i)  =>  grad_in_i = y_i (g_i - sum_j g_j y_j).
void softmax_vjp_row(const double* y, const double* g, double* gin, size_t n) {
  double dot = 0.0;
  for (size_t j = 0; j < n; ++j) dot += g[j] * y[j];
  for (size_t i = 0; i < n; ++i) gin[i] = y[i] * (g[i] - dot);
}

// ---------------------------------------------------------------- the quantiser

// Eq. 8 with N = 4 on one row, specified in correctly rounded binary32:
//   d = mx (-) mn;  s = d (/) 15;  inv = 15 (/) d;
//   t_i = (v_i (-) mn) (x) inv;  q_i = clamp(round_half_even(t_i), 0, 15).
// Multiplying by inv = 15/d (rather than dividing by the rounded s) keeps the exact
// tie at the centre of a [-2, 2] row (v = 0, t = 7.5) a tie.  A constant row
// (d == 0) gets all-zero codes and s = 0, so that dequantisation returns mn.
void quantize_row_levels(const float* v, size_t n, int levels, uint8_t* q, float* mn_out, float* s_out) {
  float mn = v[0], mx = v[0];
  for (size_t i = 1; i < n; ++i) {
    mn = std::min(mn, v[i]);
    mx = std::max(mx, v[i]);
  }
  float d = mx - mn;
  *mn_out = mn;
  if (d == 0.0f) {
    for (size_t i = 0; i < n; ++i) q[i] = 0;
    *s_out = 0.0f;
    return;
  }
  float s = d / (float)levels;
  float inv = (float)levels / d;
  for (size_t i = 0; i < n; ++i) {
    float t = (v[i] - mn) * inv;
    float r = std::nearbyintf(t);  // ties-to-even under the default rounding mode
    if (r < 0.0f) r = 0.0f;
    if (r > (float)levels) r = (float)levels;
    q[i] = (uint8_t)r;
  }
  *s_out = s;
}

void quantize_row(const float* v, size_t n, uint8_t* q, float* mn_out, float* s_out) {
  quantize_row_levels(v, n, kLevels, q, mn_out, s_out);
}

// Eq. 8 evaluated as printed, in binary64: q = round((v - min) / s), s = (max-min)/15.
// Used only to count where the binary32-specified codes above depart from it.
void quantize_row_definition(const float* v, size_t n, uint8_t* q) {
  double mn = v[0], mx = v[0];
  for (size_t i = 1; i < n; ++i) {
    mn = std::min(mn, (double)v[i]);
    mx = std::max(mx, (double)v[i]);
  }
  double s = (mx - mn) / (double)kLevels;
  for (size_t i = 0; i < n; ++i) {
    if (s == 0.0) { q[i] = 0; continue; }
    double r = std::nearbyint(((double)v[i] - mn) / s);
    r = std::min(std::max(r, 0.0), (double)kLevels);
    q[i] = (uint8_t)r;
  }
}

// Two 4-bit codes per byte over the FLAT element index e of the whole tensor:
// even e -> low nibble of byte e/2, odd e -> high nibble.  An unpaired last nibble
// leaves the high nibble zero.  (The paper fixes only "N bits per value".)
void pack_codes(const uint8_t* q, size_t n, uint8_t* bytes) {
  for (size_t b = 0; b < (n + 1) / 2; ++b) bytes[b] = 0;
  for (size_t e = 0; e < n; ++e) {
    if ((e & 1) == 0) bytes[e >> 1] |= (uint8_t)(q[e] & 0xF);
    else bytes[e >> 1] |= (uint8_t)((q[e] & 0xF) << 4);
  }
}

void unpack_codes(const uint8_t* bytes, size_t n, uint8_t* q) {
  for (size_t e = 0; e < n; ++e) {
    uint8_t b = bytes[e >> 1];
    q[e] = (e & 1) ? (uint8_t)(b >> 4) : (uint8_t)(b & 0xF);
  }
}

// General bit width N in {1, 2, 4, 8} (Eq. 8 is stated for any N): element e owns bits
// [(e N) mod 8, (e N) mod 8 + N) of byte (e N) / 8, least significant first -- for N = 4
// this is the nibble layout above.
void pack_codes_bits(const uint8_t* q, size_t n, int bits, uint8_t* bytes) {
  for (size_t b = 0; b < (n * bits + 7) / 8; ++b) bytes[b] = 0;
  for (size_t e = 0; e < n; ++e) {
    size_t bit = e * (size_t)bits;
    bytes[bit >> 3] |= (uint8_t)((q[e] & ((1u << bits) - 1u)) << (bit & 7));
  }
}

void unpack_codes_bits(const uint8_t* bytes, size_t n, int bits, uint8_t* q) {
  for (size_t e = 0; e < n; ++e) {
    size_t bit = e * (size_t)bits;
    q[e] = (uint8_t)((bytes[bit >> 3] >> (bit & 7)) & ((1u << bits) - 1u));
  }
}

bool bad_bits(int bits) { return bits != 1 && bits != 2 && bits != 4 && bits != 8; }

// Eq. 9: v_hat = q * s + min, in binary64 from the stored binary32 (min, s).
double dequantize(uint8_t q, float mn, float s) { return (double)q * (double)s + (double)mn; }

// ---------------------------------------------------------------- row-parallel driver

// Rows are independent; threads > 1 only splits the row range, the per-row code is
// the same.  Used by the benchmark's CPU-baseline leg.
template <class F>
void for_rows(size_t rows, int threads, F f) {
  if (threads <= 1 || rows < 2) {
    for (size_t r = 0; r < rows; ++r) f(r);
    return;
  }
  size_t T = std::min<size_t>((size_t)threads, rows);
  std::vector<std::thread> pool;
  for (size_t t = 0; t < T; ++t) {
    size_t lo = rows * t / T, hi = rows * (t + 1) / T;
    pool.emplace_back([=]() { for (size_t r = lo; r < hi; ++r) f(r); });
  }
  for (auto& th : pool) th.join();
}

bool bad_shape(size_t n, size_t L) { return L == 0 || (n % L) != 0; }

}  // namespace

extern "C" {

// ---- scalar / row building blocks (exposed for the pins) -------------------------
double s2a_oracle_gelu(double x) { return gelu(x); }
double s2a_oracle_gelu_grad_exact(double x) { return gelu_grad_exact(x); }
double s2a_oracle_gelu_grad_sine(double x) { return gelu_grad_sine(x); }
void s2a_oracle_softmax_row(const double* x, double* y, size_t n) { softmax_row(x, y, n); }
void s2a_oracle_softmax_vjp_row(const double* y, const double* g, double* gin, size_t n) {
  softmax_vjp_row(y, g, gin, n);
}
void s2a_oracle_quantize_row(const float* v, size_t n, uint8_t* q, float* mn, float* s) {
  quantize_row(v, n, q, mn, s);
}
void s2a_oracle_quantize_row_definition(const float* v, size_t n, uint8_t* q) {
  quantize_row_definition(v, n, q);
}
void s2a_oracle_pack(const uint8_t* q, size_t n, uint8_t* bytes) { pack_codes(q, n, bytes); }
void s2a_oracle_unpack(const uint8_t* bytes, size_t n, uint8_t* q) { unpack_codes(bytes, n, q); }
double s2a_oracle_dequantize(uint8_t q, float mn, float s) { return dequantize(q, mn, s); }
uint16_t s2a_oracle_round_bf16(double d) { return round_to_bf16_bits(d); }
float s2a_oracle_bf16_to_float(uint16_t b) { return bf16_bits_to_float(b); }

// ---- GELU forward: Eq. 10, then the clipped input is quantised (Section 3.2,
// "GeLU layer": clip to [-2, 2], then Eq. 8 over the row, on x rather than y).
// y may alias x.  meta[2r] = min, meta[2r+1] = s of row r.  Returns 0, or 2 on a
// bad shape.
int s2a_oracle_gelu_fwd(const void* x, void* y, uint8_t* codes, float* meta, size_t n,
                        size_t L, int dt, int threads) {
  if (n == 0) return 0;
  if (bad_shape(n, L)) return 2;
  std::vector<uint8_t> q(n);
  for_rows(n / L, threads, [&](size_t r) {
    std::vector<float> c(L);
    for (size_t i = 0; i < L; ++i) {
      double xi = load_elem(x, r * L + i, dt);
      c[i] = (float)std::min(std::max(xi, -2.0), 2.0);  // exact: xi is binary32/bf16
      store_elem(y, r * L + i, dt, gelu(xi));
    }
    quantize_row(c.data(), L, &q[r * L], &meta[2 * r], &meta[2 * r + 1]);
  });
  pack_codes(q.data(), n, codes);
  return 0;
}

}  // extern "C"

namespace {
// ---- SiLU / Swish (Section 3.2, last sentence of "GeLU layer": the design "is also
// effective for similar non-parametric functions, such as SiLU and Swish"; the paper gives
// no constants for them).  Reading taken here: y = x * sigmoid(x); the input is clipped to
// [-C, C] with C = 2 * 1.702 (the same range of the sigmoid's argument as GELU's [-2, 2]),
// quantised per row with Eq. 8, and the backward pass evaluates the EXACT derivative
// sigmoid(x)(1 + x(1 - sigmoid(x))) at the dequantised input.
const double kSiluClip = (double)(2.0f * 1.702f);

double silu(double x) { return x * sigmoid(x); }
double silu_grad(double x) {
  double s = sigmoid(x);
  return s * (1.0 + x * (1.0 - s));
}
}  // namespace

extern "C" {
double s2a_oracle_silu(double x) { return silu(x); }
double s2a_oracle_silu_grad(double x) { return silu_grad(x); }

int s2a_oracle_silu_fwd(const void* x, void* y, uint8_t* codes, float* meta, size_t n, size_t L, int dt,
                        int threads) {
  if (n == 0) return 0;
  if (bad_shape(n, L)) return 2;
  std::vector<uint8_t> q(n);
  for_rows(n / L, threads, [&](size_t r) {
    std::vector<float> c(L);
    for (size_t i = 0; i < L; ++i) {
      double xi = load_elem(x, r * L + i, dt);
      c[i] = (float)std::min(std::max(xi, -kSiluClip), kSiluClip);  // exact: the bound is binary32
      store_elem(y, r * L + i, dt, silu(xi));
    }
    quantize_row(c.data(), L, &q[r * L], &meta[2 * r], &meta[2 * r + 1]);
  });
  pack_codes(q.data(), n, codes);
  return 0;
}

int s2a_oracle_silu_bwd(const void* g, const uint8_t* codes, const float* meta, void* gin, size_t n, size_t L,
                        int dt, int threads) {
  if (n == 0) return 0;
  if (bad_shape(n, L)) return 2;
  std::vector<uint8_t> q(n);
  unpack_codes(codes, n, q.data());
  for_rows(n / L, threads, [&](size_t r) {
    float mn = meta[2 * r], s = meta[2 * r + 1];
    for (size_t i = 0; i < L; ++i) {
      double xh = dequantize(q[r * L + i], mn, s);
      store_elem(gin, r * L + i, dt, load_elem(g, r * L + i, dt) * silu_grad(xh));
    }
  });
  return 0;
}

// ---- GELU forward, per-TENSOR range: the other reading of Section 3.2, "GeLU layer", which
// quantises the clipped input over its min-to-max range without saying over which elements:
// here Eq. 8's min and max are taken over the whole clipped tensor instead of over each row.  Every row's metadata carries the same
// (min, s), so the backward pass is unchanged.
int s2a_oracle_gelu_fwd_tensor_range(const void* x, void* y, uint8_t* codes, float* meta, size_t n,
                                     size_t L, int dt) {
  if (n == 0) return 0;
  if (bad_shape(n, L)) return 2;
  std::vector<float> c(n);
  std::vector<uint8_t> q(n);
  for (size_t e = 0; e < n; ++e) {
    double xe = load_elem(x, e, dt);
    c[e] = (float)std::min(std::max(xe, -2.0), 2.0);
    store_elem(y, e, dt, gelu(xe));
  }
  float mn, s;
  quantize_row(c.data(), n, q.data(), &mn, &s);  // one "row": the whole tensor
  for (size_t r = 0; r < n / L; ++r) {
    meta[2 * r] = mn;
    meta[2 * r + 1] = s;
  }
  pack_codes(q.data(), n, codes);
  return 0;
}

// ---- GELU backward: Eq. 9 then Eq. 12 at x_hat, times grad_out.
int s2a_oracle_gelu_bwd(const void* g, const uint8_t* codes, const float* meta, void* gin,
                        size_t n, size_t L, int dt, int threads) {
  if (n == 0) return 0;
  if (bad_shape(n, L)) return 2;
  std::vector<uint8_t> q(n);
  unpack_codes(codes, n, q.data());
  for_rows(n / L, threads, [&](size_t r) {
    float mn = meta[2 * r], s = meta[2 * r + 1];
    for (size_t i = 0; i < L; ++i) {
      double xh = dequantize(q[r * L + i], mn, s);
      double gi = load_elem(g, r * L + i, dt);
      store_elem(gin, r * L + i, dt, gi * gelu_grad_sine(xh));
    }
  });
  return 0;
}

// ---- Softmax forward: Eq. 7 per row, output rounded to the I/O type; the values
// AS WRITTEN are then quantised with Eq. 8 over the row.
int s2a_oracle_softmax_fwd(const void* x, void* y, uint8_t* codes, float* meta, size_t n,
                           size_t L, int dt, int threads) {
  if (n == 0) return 0;
  if (bad_shape(n, L)) return 2;
  std::vector<uint8_t> q(n);
  for_rows(n / L, threads, [&](size_t r) {
    std::vector<double> xr(L), yr(L);
    std::vector<float> v(L);
    for (size_t i = 0; i < L; ++i) xr[i] = load_elem(x, r * L + i, dt);
    softmax_row(xr.data(), yr.data(), L);
    for (size_t i = 0; i < L; ++i) v[i] = store_elem(y, r * L + i, dt, yr[i]);
    quantize_row(v.data(), L, &q[r * L], &meta[2 * r], &meta[2 * r + 1]);
  });
  pack_codes(q.data(), n, codes);
  return 0;
}

// ---- Softmax backward: Eq. 9, then the Jacobian of Eq. 7 evaluated at y_hat.
int s2a_oracle_softmax_bwd(const void* g, const uint8_t* codes, const float* meta, void* gin,
                           size_t n, size_t L, int dt, int threads) {
  if (n == 0) return 0;
  if (bad_shape(n, L)) return 2;
  std::vector<uint8_t> q(n);
  unpack_codes(codes, n, q.data());
  for_rows(n / L, threads, [&](size_t r) {
    float mn = meta[2 * r], s = meta[2 * r + 1];
    std::vector<double> yh(L), gr(L), out(L);
    for (size_t i = 0; i < L; ++i) {
      yh[i] = dequantize(q[r * L + i], mn, s);
      gr[i] = load_elem(g, r * L + i, dt);
    }
    softmax_vjp_row(yh.data(), gr.data(), out.data(), L);
    for (size_t i = 0; i < L; ++i) store_elem(gin, r * L + i, dt, out[i]);
  });
  return 0;
}

// ---- The four kernels at a general bit width N (Eq. 8 with 2^N - 1 levels); N = 4
// reproduces the functions above bit for bit.  kind: 0 GELU, 1 softmax.
int s2a_oracle_fwd_bits(int kind, const void* x, void* y, uint8_t* codes, float* meta, size_t n, size_t L,
                        int bits, int dt) {
  if (n == 0) return 0;
  if (bad_shape(n, L) || bad_bits(bits)) return 2;
  const int levels = (1 << bits) - 1;
  std::vector<uint8_t> q(n);
  for (size_t r = 0; r < n / L; ++r) {
    std::vector<float> v(L);
    if (kind == 0) {
      for (size_t i = 0; i < L; ++i) {
        double xi = load_elem(x, r * L + i, dt);
        v[i] = (float)std::min(std::max(xi, -2.0), 2.0);
        store_elem(y, r * L + i, dt, gelu(xi));
      }
    } else {
      std::vector<double> xr(L), yr(L);
      for (size_t i = 0; i < L; ++i) xr[i] = load_elem(x, r * L + i, dt);
      softmax_row(xr.data(), yr.data(), L);
      for (size_t i = 0; i < L; ++i) v[i] = store_elem(y, r * L + i, dt, yr[i]);
    }
    quantize_row_levels(v.data(), L, levels, &q[r * L], &meta[2 * r], &meta[2 * r + 1]);
  }
  pack_codes_bits(q.data(), n, bits, codes);
  return 0;
}

int s2a_oracle_bwd_bits(int kind, const void* g, const uint8_t* codes, const float* meta, void* gin, size_t n,
                        size_t L, int bits, int dt) {
  if (n == 0) return 0;
  if (bad_shape(n, L) || bad_bits(bits)) return 2;
  std::vector<uint8_t> q(n);
  unpack_codes_bits(codes, n, bits, q.data());
  for (size_t r = 0; r < n / L; ++r) {
    float mn = meta[2 * r], s = meta[2 * r + 1];
    if (kind == 0) {
      for (size_t i = 0; i < L; ++i)
        store_elem(gin, r * L + i, dt,
                   load_elem(g, r * L + i, dt) * gelu_grad_sine(dequantize(q[r * L + i], mn, s)));
    } else {
      std::vector<double> yh(L), gr(L), out(L);
      for (size_t i = 0; i < L; ++i) {
        yh[i] = dequantize(q[r * L + i], mn, s);
        gr[i] = load_elem(g, r * L + i, dt);
      }
      softmax_vjp_row(yh.data(), gr.data(), out.data(), L);
      for (size_t i = 0; i < L; ++i) store_elem(gin, r * L + i, dt, out[i]);
    }
  }
  return 0;
}

void s2a_oracle_quantize_row_levels(const float* v, size_t n, int levels, uint8_t* q, float* mn, float* s) {
  quantize_row_levels(v, n, levels, q, mn, s);
}
void s2a_oracle_pack_bits(const uint8_t* q, size_t n, int bits, uint8_t* bytes) { pack_codes_bits(q, n, bits, bytes); }
void s2a_oracle_unpack_bits(const uint8_t* bytes, size_t n, int bits, uint8_t* q) {
  unpack_codes_bits(bytes, n, bits, q);
}

// ---- Quantise an already materialised tensor row by row (Eq. 8 + packing); lets a
// test check that stored codes are exactly Q(values as written).
int s2a_oracle_quantize_tensor(const void* v, uint8_t* codes, float* meta, size_t n, size_t L,
                               int dt, int threads) {
  if (n == 0) return 0;
  if (bad_shape(n, L)) return 2;
  std::vector<uint8_t> q(n);
  for_rows(n / L, threads, [&](size_t r) {
    std::vector<float> c(L);
    for (size_t i = 0; i < L; ++i) {
      c[i] = (float)load_elem(v, r * L + i, dt);
    }
    quantize_row(c.data(), L, &q[r * L], &meta[2 * r], &meta[2 * r + 1]);
  });
  pack_codes(q.data(), n, codes);
  return 0;
}

// ---- ReLU (Section 3.2, "ReLU layer"): the derivative takes the values 0 and 1 only, so
// the stash is one bit per element: 1 where x > 0.  Bit (e mod 8) of byte e / 8, least
// significant bit first, over the flat element index; unused bits of the last byte are 0.
// Forward: y = x where x > 0, else +0.  Backward: grad_in = grad_out where the bit is set,
// else +0.
int s2a_oracle_relu_fwd(const void* x, void* y, uint8_t* mask, size_t n, int dt) {
  for (size_t b = 0; b < (n + 7) / 8; ++b) mask[b] = 0;
  for (size_t e = 0; e < n; ++e) {
    double xe = load_elem(x, e, dt);
    bool pos = xe > 0.0;
    store_elem(y, e, dt, pos ? xe : 0.0);
    if (pos) mask[e >> 3] |= (uint8_t)(1u << (e & 7));
  }
  return 0;
}

int s2a_oracle_relu_bwd(const void* g, const uint8_t* mask, void* gin, size_t n, int dt) {
  for (size_t e = 0; e < n; ++e) {
    bool pos = (mask[e >> 3] >> (e & 7)) & 1;
    store_elem(gin, e, dt, pos ? load_elem(g, e, dt) : 0.0);
  }
  return 0;
}

// ---- Channel Average Pooling (Eq. 5): y_k = (1/r) sum_{j<r} x_{k r + j} along the channel
// axis of an [n_rows, channels] tensor; backward: dL/dx_{k r + j} = (1/r) dL/dy_k.
int s2a_oracle_cap_fwd(const void* x, void* y, size_t n_rows, size_t channels, size_t r, int dt) {
  if (r == 0 || channels % r != 0) return 2;
  const size_t out_ch = channels / r;
  for (size_t row = 0; row < n_rows; ++row)
    for (size_t k = 0; k < out_ch; ++k) {
      double sum = 0.0;
      for (size_t j = 0; j < r; ++j) sum += load_elem(x, row * channels + k * r + j, dt);
      store_elem(y, row * out_ch + k, dt, sum / (double)r);
    }
  return 0;
}

int s2a_oracle_cap_bwd(const void* g, void* gin, size_t n_rows, size_t channels, size_t r, int dt) {
  if (r == 0 || channels % r != 0) return 2;
  const size_t out_ch = channels / r;
  for (size_t row = 0; row < n_rows; ++row)
    for (size_t k = 0; k < out_ch; ++k) {
      double v = load_elem(g, row * out_ch + k, dt) / (double)r;
      for (size_t j = 0; j < r; ++j) store_elem(gin, row * channels + k * r + j, dt, v);
    }
  return 0;
}

// ---- Low-Rank Prompt, forward (Eq. 3): y = x + A B with A [tokens, rank], B [rank, channels]
// (binary32 parameters), the same prompt added to every sample of the batch.  Backward to
// the activation (Eq. 4) is the identity and needs no kernel.
int s2a_oracle_lrp_fwd(const void* x, const float* A, const float* B, void* y, size_t batch, size_t tokens,
                       size_t channels, size_t rank, int dt) {
  for (size_t b = 0; b < batch; ++b)
    for (size_t t = 0; t < tokens; ++t)
      for (size_t c = 0; c < channels; ++c) {
        double p = 0.0;
        for (size_t k = 0; k < rank; ++k) p += (double)A[t * rank + k] * (double)B[k * channels + c];
        size_t e = (b * tokens + t) * channels + c;
        store_elem(y, e, dt, load_elem(x, e, dt) + p);
      }
  return 0;
}

// Number of hardware threads the row-parallel driver can use.
int s2a_oracle_hardware_threads() {
  unsigned h = std::thread::hardware_concurrency();
  return h == 0 ? 1 : (int)h;
}

}  // extern "C"
