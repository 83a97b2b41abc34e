// CPU oracle for the W4A4 + low-rank linear forward.   TEST INFRASTRUCTURE ONLY.
//
// Plain, single-threaded, deliberately slow C++17 written from the paper's equations.  It exists
// so that the CUDA path can be checked element by element; it is never part of the product path,
// shares no code, header, table or helper with the CUDA sources, and is only ever called from the
// tests, the smoke check and the benchmark's CPU-baseline leg.
//
// Compile with:  g++ -O2 -std=c++17 -ffp-contract=off -fno-fast-math  (no FMA contraction: every
// FP32 operation below is a separately rounded IEEE operation, in exactly the order written).
//
// What it computes, per token row m and 64-channel group g (K = C_in, N = C_out, G = K/64):
//
//   Eq. 5   smoothing            rl[k]   = 1.0f / lambda[k]                      (FP32 divide)
//                                xh[m,k] = f32(X[m,k]) * rl[k]                   (one FP32 multiply)
//   Eq. 8   clip threshold       a[m,g]  = max_k |xh[m,k]|  over the group       (exact)
//                                u       = rho * a[m,g]                          (FP32 multiply)
//   Eq. 9/4 activation scale     s[m,g]  = u / 7.0f                              (FP32 divide); a == 0 -> s = 0
//   Eq. 3   quantizer, z0 = 0    is      = 1.0f / s[m,g]                         (FP32 divide)
//                                q[m,k]  = clip(rint(xh[m,k] * is), -8, 7)       (FP32 multiply, round half to even)
//   Eq. 7   low-rank branch      T[m,j]  = f32( sum_k f64(bf16(xh[m,k])) * f64(L1[k,j]) )      k ascending
//   Eq. 7   4-bit branch         P[m,g,n]= sum_{k in g} q[m,k] * qw[k,n]                       (int32, exact)
//   Eq. 7/11 assembly            Y[m,n]  = sum_g f64(P) * f64(s[m,g]) * f64(sw[g,n])           g ascending
//                                        + sum_j f64(T[m,j]) * f64(L2[j,n])                    j ascending
//                                        + f64(b[n])
//   The dequantisation factor of Eq. 3 (the leading "s *") is what turns P into a real number:
//   one factor from the activation side (s) and one from the weight side (sw).
//
// rho is the clipping ratio fetched from the (expert, layer, timestep-bin) table (Sec. III-C); the
// reference magnitude m_{l,k} of Eq. 8 is taken dynamically as the group's absolute maximum.
//
// Readings where the paper is silent: INT4
// two's complement codes, q_max = 7 for the scale and [-8, 7] for the clip, ties to even, group 64,
// multiplication by a reciprocal in place of the division inside Eq. 3, bias added at the end.
//
// The second half of the file holds the MXFP4 variant of the layer (its own header comment).
//
// Parity status: every function below is pinned by tests that do not come from this file
// (on-grid round trips, tie cases, saturation, brute-force dot products, the r = 0 and
// "quantization disabled" reductions to a plain FP64 matrix product).  The paper prints no worked
// numbers for this path, so nothing here is pinned against the authors' own code.

#include <algorithm>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <vector>

namespace {

constexpr int kGroup = 64;

inline float bf16_to_f32(uint16_t h) {
  uint32_t u = static_cast<uint32_t>(h) << 16;
  float f;
  std::memcpy(&f, &u, sizeof(f));
  return f;
}

// FP32 -> BF16, round to nearest, ties to even.  NaN stays NaN (quiet).
inline uint16_t f32_to_bf16_rne(float f) {
  uint32_t u;
  std::memcpy(&u, &f, sizeof(u));
  if ((u & 0x7fffffffu) > 0x7f800000u) return static_cast<uint16_t>((u >> 16) | 0x0040u);
  const uint32_t lsb = (u >> 16) & 1u;
  u += 0x7fffu + lsb;
  return static_cast<uint16_t>(u >> 16);
}

// Eq. 5: one smoothed activation, FP32.
inline float smooth(uint16_t x_bits, float rl) { return bf16_to_f32(x_bits) * rl; }

// Smooth + quantize one row.  q: K codes, s: G scales.  xh_out (optional): K smoothed values.
void quantize_row(const uint16_t* x, const float* rl, float rho, int K, int8_t* q, float* s, float* xh_out) {
  std::vector<float> xh(static_cast<size_t>(K));
  for (int k = 0; k < K; ++k) xh[k] = smooth(x[k], rl[k]);
  const int G = K / kGroup;
  for (int g = 0; g < G; ++g) {
    const float* v = xh.data() + static_cast<size_t>(g) * kGroup;
    float a = 0.0f;
    for (int i = 0; i < kGroup; ++i) {
      const float t = std::fabs(v[i]);
      if (t > a) a = t;
    }
    int8_t* qg = q + static_cast<size_t>(g) * kGroup;
    if (!(a > 0.0f)) {
      s[g] = 0.0f;
      for (int i = 0; i < kGroup; ++i) qg[i] = 0;
      continue;
    }
    const float u = rho * a;     // Eq. 8
    const float sc = u / 7.0f;   // Eq. 9 with q_max = 7
    const float is = 1.0f / sc;
    s[g] = sc;
    for (int i = 0; i < kGroup; ++i) {
      const float z = v[i] * is;            // Eq. 3: z / s as a multiply by the reciprocal
      float rz = std::nearbyintf(z);        // default rounding mode: nearest, ties to even
      if (rz < -8.0f) rz = -8.0f;
      if (rz > 7.0f) rz = 7.0f;
      qg[i] = static_cast<int8_t>(static_cast<int>(rz));
    }
  }
  if (xh_out) std::memcpy(xh_out, xh.data(), sizeof(float) * static_cast<size_t>(K));
}

void reciprocal_lambda(const float* lambda, int K, std::vector<float>& rl) {
  rl.resize(static_cast<size_t>(K));
  for (int k = 0; k < K; ++k) rl[k] = 1.0f / lambda[k];
}

// Eq. 7, first factor of the low-rank branch, one row.  L1 is K x r BF16 row-major.
void lowrank_down_row(const uint16_t* x, const float* rl, const uint16_t* L1, int K, int r, float* T) {
  std::vector<double> acc(static_cast<size_t>(r), 0.0);
  for (int k = 0; k < K; ++k) {
    const float xh = smooth(x[k], rl[k]);
    const double xb = static_cast<double>(bf16_to_f32(f32_to_bf16_rne(xh)));
    const uint16_t* l = L1 + static_cast<size_t>(k) * r;
    for (int j = 0; j < r; ++j) acc[j] += xb * static_cast<double>(bf16_to_f32(l[j]));
  }
  for (int j = 0; j < r; ++j) T[j] = static_cast<float>(acc[j]);
}

// Eq. 7, 4-bit branch, one row: P[g][n] for all groups.  qw is K x N int8 row-major.
void partials_row(const int8_t* q, const int8_t* qw, int K, int N, int32_t* P) {
  const int G = K / kGroup;
  for (int g = 0; g < G; ++g) {
    int32_t* p = P + static_cast<size_t>(g) * N;
    for (int n = 0; n < N; ++n) p[n] = 0;
    for (int i = 0; i < kGroup; ++i) {
      const int k = g * kGroup + i;
      const int32_t a = q[k];
      const int8_t* w = qw + static_cast<size_t>(k) * N;
      for (int n = 0; n < N; ++n) p[n] += a * static_cast<int32_t>(w[n]);
    }
  }
}

// Eq. 7 / 11 assembly, one row.
void assemble_row(const int32_t* P, const float* s, const float* sw, const float* T, const uint16_t* L2,
                  const float* bias, int K, int N, int r, double* Y) {
  const int G = K / kGroup;
  for (int n = 0; n < N; ++n) {
    double y = 0.0;
    for (int g = 0; g < G; ++g) {
      y += static_cast<double>(P[static_cast<size_t>(g) * N + n]) * static_cast<double>(s[g]) *
           static_cast<double>(sw[static_cast<size_t>(g) * N + n]);
    }
    for (int j = 0; j < r; ++j) {
      y += static_cast<double>(T[j]) * static_cast<double>(bf16_to_f32(L2[static_cast<size_t>(j) * N + n]));
    }
    if (bias) y += static_cast<double>(bias[n]);
    Y[n] = y;
  }
}

}  // namespace

extern "C" {

// Eq. 3-5, 8-9.  X: M x K BF16 bit patterns; q: M x K codes; s: M x (K/64) scales.  xh (nullable): M x K.
int oracle_quantize(const uint16_t* X, const float* lambda, float rho, int M, int K, int8_t* q, float* s,
                    float* xh) {
  if (K <= 0 || K % kGroup != 0 || M < 0) return 1;
  std::vector<float> rl;
  reciprocal_lambda(lambda, K, rl);
  const int G = K / kGroup;
  for (int m = 0; m < M; ++m) {
    quantize_row(X + static_cast<size_t>(m) * K, rl.data(), rho, K, q + static_cast<size_t>(m) * K,
                 s + static_cast<size_t>(m) * G, xh ? xh + static_cast<size_t>(m) * K : nullptr);
  }
  return 0;
}

// Eq. 7 (X-hat L1).  T: M x r FP32.
int oracle_lowrank_down(const uint16_t* X, const float* lambda, const uint16_t* L1, int M, int K, int r, float* T) {
  if (K <= 0 || M < 0 || r < 0) return 1;
  std::vector<float> rl;
  reciprocal_lambda(lambda, K, rl);
  for (int m = 0; m < M; ++m) {
    lowrank_down_row(X + static_cast<size_t>(m) * K, rl.data(), L1, K, r, T + static_cast<size_t>(m) * r);
  }
  return 0;
}

// Eq. 7 (Q_A(X-hat) R-hat as integers).  q: M x K, qw: K x N, P: M x G x N int32.
int oracle_partials(const int8_t* q, const int8_t* qw, int M, int K, int N, int32_t* P) {
  if (K <= 0 || K % kGroup != 0) return 1;
  const int G = K / kGroup;
  for (int m = 0; m < M; ++m) {
    partials_row(q + static_cast<size_t>(m) * K, qw, K, N, P + static_cast<size_t>(m) * G * N);
  }
  return 0;
}

// Eq. 7 / 11 assembly from already computed pieces.  Y64: M x N; Ybf16 (nullable): M x N bit patterns.
int oracle_assemble(const int32_t* P, const float* s, const float* sw, const float* T, const uint16_t* L2,
                    const float* bias, int M, int K, int N, int r, double* Y64, uint16_t* Ybf16) {
  if (K <= 0 || K % kGroup != 0) return 1;
  const int G = K / kGroup;
  for (int m = 0; m < M; ++m) {
    double* y = Y64 + static_cast<size_t>(m) * N;
    assemble_row(P + static_cast<size_t>(m) * G * N, s + static_cast<size_t>(m) * G, sw,
                 r > 0 ? T + static_cast<size_t>(m) * r : nullptr, L2, bias, K, N, r, y);
    if (Ybf16) {
      for (int n = 0; n < N; ++n) Ybf16[static_cast<size_t>(m) * N + n] = f32_to_bf16_rne(static_cast<float>(y[n]));
    }
  }
  return 0;
}

// The whole layer for a chosen set of rows (rows are independent, so a row subset is exact for
// those rows).  rows[i] indexes X; outputs are indexed by i.  Any of q, s, T, P, Ybf16 may be null.
int oracle_forward_rows(const uint16_t* X, const int* rows, int num_rows, int K, int N, int r, const float* lambda,
                        float rho, const uint16_t* L1, const uint16_t* L2, const int8_t* qw, const float* sw,
                        const float* bias, int8_t* q, float* s, float* T, int32_t* P, double* Y64, uint16_t* Ybf16) {
  if (K <= 0 || K % kGroup != 0 || N <= 0 || r < 0) return 1;
  const int G = K / kGroup;
  std::vector<float> rl;
  reciprocal_lambda(lambda, K, rl);
  std::vector<int8_t> qrow(static_cast<size_t>(K));
  std::vector<float> srow(static_cast<size_t>(G));
  std::vector<float> trow(static_cast<size_t>(r > 0 ? r : 1));
  std::vector<int32_t> prow(static_cast<size_t>(G) * N);
  std::vector<double> yrow(static_cast<size_t>(N));
  for (int i = 0; i < num_rows; ++i) {
    const uint16_t* x = X + static_cast<size_t>(rows[i]) * K;
    quantize_row(x, rl.data(), rho, K, qrow.data(), srow.data(), nullptr);
    if (r > 0) lowrank_down_row(x, rl.data(), L1, K, r, trow.data());
    partials_row(qrow.data(), qw, K, N, prow.data());
    assemble_row(prow.data(), srow.data(), sw, r > 0 ? trow.data() : nullptr, L2, bias, K, N, r, yrow.data());
    if (q) std::memcpy(q + static_cast<size_t>(i) * K, qrow.data(), static_cast<size_t>(K));
    if (s) std::memcpy(s + static_cast<size_t>(i) * G, srow.data(), sizeof(float) * G);
    if (T && r > 0) std::memcpy(T + static_cast<size_t>(i) * r, trow.data(), sizeof(float) * r);
    if (P) std::memcpy(P + static_cast<size_t>(i) * G * N, prow.data(), sizeof(int32_t) * static_cast<size_t>(G) * N);
    if (Y64) std::memcpy(Y64 + static_cast<size_t>(i) * N, yrow.data(), sizeof(double) * N);
    if (Ybf16) {
      for (int n = 0; n < N; ++n) Ybf16[static_cast<size_t>(i) * N + n] = f32_to_bf16_rne(static_cast<float>(yrow[n]));
    }
  }
  return 0;
}

// Eq. 5-7 with both quantizers switched off, everything in FP64:
//   Y = (X D^-1) L1 L2 + (X D^-1) R + b,   X-hat by true division.
// With R = D W - L1 L2 this must reproduce X W (Eq. 1) to round-off.
int oracle_forward_noquant(const double* X, const double* lambda, const double* L1, const double* L2, const double* R,
                           const double* bias, int M, int K, int N, int r, double* Y) {
  std::vector<double> xh(static_cast<size_t>(K));
  std::vector<double> t(static_cast<size_t>(r > 0 ? r : 1));
  for (int m = 0; m < M; ++m) {
    for (int k = 0; k < K; ++k) xh[k] = X[static_cast<size_t>(m) * K + k] / lambda[k];
    for (int j = 0; j < r; ++j) {
      double a = 0.0;
      for (int k = 0; k < K; ++k) a += xh[k] * L1[static_cast<size_t>(k) * r + j];
      t[j] = a;
    }
    for (int n = 0; n < N; ++n) {
      double y = 0.0;
      for (int k = 0; k < K; ++k) y += xh[k] * R[static_cast<size_t>(k) * N + n];
      for (int j = 0; j < r; ++j) y += t[j] * L2[static_cast<size_t>(j) * N + n];
      if (bias) y += bias[n];
      Y[static_cast<size_t>(m) * N + n] = y;
    }
  }
  return 0;
}

// BF16 conversion exposed for its own pin (compared against an independent implementation).
uint16_t oracle_f32_to_bf16(float f) { return f32_to_bf16_rne(f); }

}  // extern "C"

// =====================================================================================================
// MXFP4 variant of the same layer (the data format the paper's Table 1 says its 4-bit runs used, and the
// hardware 4-bit floating-point path that Sec. IV-D names as the way forward).  Element and scale formats and the
// conversion rule are those of the OCP Microscaling Formats (MX) specification v1.0:
//
//   block          32 consecutive input channels of one token (activations) / of one output column (weights)
//   scale          E8M0: one byte e, value 2^(e - 127)
//   element        E2M1: sign, 2 exponent bits, 1 mantissa bit: +-{0, 0.5, 1, 1.5, 2, 3, 4, 6}
//   conversion     shared exponent = floor(log2(block maximum)) - 2 (2 = exponent of the largest E2M1 binade),
//                  element = round-to-nearest-even of value / 2^shared onto the E2M1 grid, saturating at +-6
//
// The paper's clipping ratio enters exactly where Eq. 8 puts it: the block maximum is replaced by the clip
// threshold rho * max|xh| before the shared exponent is taken.
//
//   xh[m,k]   = f32(X[m,k]) * (1.0f / lambda[k])                      as in the INT4 path (Eq. 5)
//   u         = rho * max_{k in block} |xh[m,k]|                      FP32 multiply (Eq. 8)
//   e[m,b]    = max(exponent field of u - 2, 0)                       (u == 0: e = 0, all elements 0;
//                                                                      the exponent field of a subnormal u is 0)
//   a[m,k]    = E2M1_RNE_sat( xh[m,k] * 2^(127 - e[m,b]) )            exact power-of-two scaling, then rounding
//   Y[m,n]    = sum_b 2^(e[m,b]-127) 2^(ew[b,n]-127) sum_{k in b} a[m,k] w[k,n]  +  T L2  +  b     (FP64)
//
// T is the same low-rank intermediate as in the INT4 path.
// =====================================================================================================
namespace {

constexpr int kMxBlock = 32;
const float kE2M1Value[8] = {0.0f, 0.5f, 1.0f, 1.5f, 2.0f, 3.0f, 4.0f, 6.0f};

// Round to nearest E2M1 value, ties to the code with an even mantissa bit, saturate at 6.  Returns the 4-bit code
// (bit 3 = sign, taken from v even when the magnitude rounds to zero).
inline uint8_t e2m1_rne_sat(float v) {
  const uint8_t sign = std::signbit(v) ? 8u : 0u;
  const float a = std::fabs(v);
  int idx = 7;
  for (int i = 0; i < 7; ++i) {
    const float lo = kE2M1Value[i], hi = kE2M1Value[i + 1];
    if (a < hi) {
      const float mid = 0.5f * (lo + hi);  // exact
      if (a < mid) idx = i;
      else if (a > mid) idx = i + 1;
      else idx = (i % 2 == 0) ? i : i + 1;  // tie: the code whose last bit is 0
      break;
    }
  }
  return static_cast<uint8_t>(sign | idx);
}

inline double e2m1_value(uint8_t code) {
  const double v = kE2M1Value[code & 7];
  return (code & 8) ? -v : v;
}

inline uint32_t f32_bits(float f) {
  uint32_t u;
  std::memcpy(&u, &f, sizeof(u));
  return u;
}

// One row: codes[K] (one E2M1 code per byte), exps[K/32] (E8M0 bytes).
void mx_quantize_row(const uint16_t* x, const float* rl, float rho, int K, uint8_t* codes, uint8_t* exps) {
  for (int b = 0; b < K / kMxBlock; ++b) {
    float xh[kMxBlock];
    float a = 0.0f;
    for (int i = 0; i < kMxBlock; ++i) {
      xh[i] = smooth(x[b * kMxBlock + i], rl[b * kMxBlock + i]);
      const float t = std::fabs(xh[i]);
      if (t > a) a = t;
    }
    const float u = rho * a;
    const int field = static_cast<int>((f32_bits(u) >> 23) & 0xffu);
    const int e = field > 2 ? field - 2 : 0;
    exps[b] = static_cast<uint8_t>(e);
    const float inv = std::ldexp(1.0f, 127 - e);  // 2^(127 - e), a normal FP32 number for every e in [0, 252]
    for (int i = 0; i < kMxBlock; ++i) {
      codes[b * kMxBlock + i] = (a > 0.0f) ? e2m1_rne_sat(xh[i] * inv) : 0;
    }
  }
}

}  // namespace

extern "C" {

// MXFP4 activation quantization of every row.  codes: M x K, exps: M x K/32.
int oracle_mx_quantize(const uint16_t* X, const float* lambda, float rho, int M, int K, uint8_t* codes, uint8_t* exps) {
  if (K <= 0 || K % kMxBlock != 0 || M < 0) return 1;
  std::vector<float> rl;
  reciprocal_lambda(lambda, K, rl);
  for (int m = 0; m < M; ++m) {
    mx_quantize_row(X + static_cast<size_t>(m) * K, rl.data(), rho, K, codes + static_cast<size_t>(m) * K,
                    exps + static_cast<size_t>(m) * (K / kMxBlock));
  }
  return 0;
}

// The E2M1 rounding on its own, for its pins.
uint8_t oracle_e2m1_rne_sat(float v) { return e2m1_rne_sat(v); }

// The whole MXFP4 layer for a chosen set of rows.  wcodes: K x N E2M1 codes (one per byte), wexps: K/32 x N E8M0.
// Any of codes, exps, T, Ybf16 may be null.
int oracle_mx_forward_rows(const uint16_t* X, const int* rows, int num_rows, int K, int N, int r, const float* lambda,
                           float rho, const uint16_t* L1, const uint16_t* L2, const uint8_t* wcodes,
                           const uint8_t* wexps, const float* bias, uint8_t* codes, uint8_t* exps, float* T,
                           double* Y64, uint16_t* Ybf16) {
  if (K <= 0 || K % kMxBlock != 0 || N <= 0 || r < 0) return 1;
  const int B = K / kMxBlock;
  std::vector<float> rl;
  reciprocal_lambda(lambda, K, rl);
  std::vector<uint8_t> crow(static_cast<size_t>(K)), erow(static_cast<size_t>(B));
  std::vector<float> trow(static_cast<size_t>(r > 0 ? r : 1));
  std::vector<double> yrow(static_cast<size_t>(N)), dot(static_cast<size_t>(N));
  for (int i = 0; i < num_rows; ++i) {
    const uint16_t* x = X + static_cast<size_t>(rows[i]) * K;
    mx_quantize_row(x, rl.data(), rho, K, crow.data(), erow.data());
    if (r > 0) lowrank_down_row(x, rl.data(), L1, K, r, trow.data());
    // Every output channel n sums its blocks b in ascending order, and inside a block its 32 products in
    // ascending k; the loops run with n innermost only so that the [K, N] weight arrays are read along rows.
    std::fill(yrow.begin(), yrow.end(), 0.0);
    for (int b = 0; b < B; ++b) {
      std::fill(dot.begin(), dot.end(), 0.0);  // multiples of 0.25, at most 32 * 36: exact
      for (int j = 0; j < kMxBlock; ++j) {
        const int k = b * kMxBlock + j;
        const double a = e2m1_value(crow[k]);
        for (int n = 0; n < N; ++n) dot[n] += a * e2m1_value(wcodes[static_cast<size_t>(k) * N + n]);
      }
      const double sa = std::ldexp(1.0, static_cast<int>(erow[b]) - 127);
      for (int n = 0; n < N; ++n) {
        yrow[n] += dot[n] * sa * std::ldexp(1.0, static_cast<int>(wexps[static_cast<size_t>(b) * N + n]) - 127);
      }
    }
    for (int n = 0; n < N; ++n) {
      double y = yrow[n];
      for (int j = 0; j < r; ++j) {
        y += static_cast<double>(trow[j]) * static_cast<double>(bf16_to_f32(L2[static_cast<size_t>(j) * N + n]));
      }
      if (bias) y += static_cast<double>(bias[n]);
      if (Y64) Y64[static_cast<size_t>(i) * N + n] = y;
      if (Ybf16) Ybf16[static_cast<size_t>(i) * N + n] = f32_to_bf16_rne(static_cast<float>(y));
    }
    if (codes) std::memcpy(codes + static_cast<size_t>(i) * K, crow.data(), static_cast<size_t>(K));
    if (exps) std::memcpy(exps + static_cast<size_t>(i) * B, erow.data(), static_cast<size_t>(B));
    if (T && r > 0) std::memcpy(T + static_cast<size_t>(i) * r, trow.data(), sizeof(float) * r);
  }
  return 0;
}

}  // extern "C"
