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
// Readings where the paper is silent are listed in the repository's design notes; in short: INT4
// two's complement codes, q_max = 7 for the scale and [-8, 7] for the clip, ties to even, group 64,
// multiplication by a reciprocal in place of the division inside Eq. 3, bias added at the end.
//
// Parity status: every function below is pinned by tests that do not come from this file
// (on-grid round trips, tie cases, saturation, brute-force dot products, the r = 0 and
// "quantization disabled" reductions to a plain FP64 matrix product).  The paper prints no worked
// numbers for this path, so nothing here is pinned against the authors' own code.

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
