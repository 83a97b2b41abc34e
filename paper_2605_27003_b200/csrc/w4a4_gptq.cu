// w4a4_gptq_quantize: GPTQ on the residual branch (Sec. III-B), entirely on the device in FP64.
//
// The published algorithm (Frantar et al., 2023, Algorithm 1 with the Cholesky reformulation of Sec. 4) quantizes
// the input channels of R [K, N] in order and spreads each channel's error, scaled by a row of
// U = chol(H^-1, upper), over the channels still to come, H = X_hat^T X_hat being the second-order statistic of the
// layer's calibration inputs.  Here:
//
//   1. H (upper triangle) = X_hat^T X_hat by a tiled FP64 GEMM; dead channels and damping on the diagonal.
//   2. U without ever forming H^-1: factor H = V V^T with V UPPER triangular (a Cholesky factorization taken from
//      the last channel to the first, blocked by 64: diagonal block, panel solve, rank-64 update), then U = V^-1
//      (blocked triangular inverse, bottom up).  H^-1 = V^-T V^-1 = U^T U with U upper and a positive diagonal,
//      which is the unique factor the algorithm asks for.
//   3. The sweep, one 64-channel group at a time: one thread per output channel holds the group's 64 weights in
//      registers, takes the group scale, quantizes channel after channel and applies the in-group updates; the
//      group's scaled errors then update all later channels by one more GEMM (the algorithm's lazy batch).
//
// Nothing here waits on another block: every dependency is a kernel boundary, on the caller's stream or on an event
// between it and one side stream of the call's own.
#include "../../include/w4a4.h"

#include <cuda_runtime.h>

#include <cstdint>

namespace {

constexpr int kNb = 64;     // block of the factorization = quantization group = lazy batch
constexpr int kBand = 512;  // columns per band of the factorization, rows per band of the triangular inverse
constexpr int kLazy = 256;  // input channels per lazy batch of the sweep

// ---------------------------------------------------------------------------------------------------------
// C[m, n] = beta * C[m, n] + alpha * sum_k A(m, k) * B(k, n), every operand addressed by two strides so that a
// transposed or sub-matrix operand costs nothing.  (16 TM) x 64 tile per block in 16-deep slices, double-buffered in
// shared memory by asynchronous copies; eight warps, each a (4 TM) x 32 corner as 8 x 8 x 4 FP64 tensor-core steps.  Structure flags: kUpperOut -- blocks whose tile lies entirely below the diagonal return at once (only the
// upper triangle of C is wanted); kAUpper -- A(m, k) = 0 for k < m, so the sum starts at the tile's first row;
// kBUpper -- B(k, n) = 0 for k > n, so the sum ends at the tile's last column.
// ---------------------------------------------------------------------------------------------------------
constexpr int kBN = 64, kBK = 16;
enum : int { kUpperOut = 1, kAUpper = 2, kBUpper = 4 };

// 8-byte asynchronous copy global -> shared; with `valid` false nothing is read and zeros are written.
__device__ __forceinline__ void async_copy8(double* smem_dst, const double* gmem_src, bool valid) {
  const unsigned dst = static_cast<unsigned>(__cvta_generic_to_shared(smem_dst));
  const int src_bytes = valid ? 8 : 0;
  asm volatile("cp.async.ca.shared.global [%0], [%1], 8, %2;" ::"r"(dst), "l"(gmem_src), "r"(src_bytes) : "memory");
}

// D (8 x 8) += A (8 x 4) B (4 x 8) on the FP64 tensor core; per lane one element of A and B, two of D.
__device__ __forceinline__ void dmma_8x8x4(double (&d)[2], double a, double b) {
  asm volatile("mma.sync.aligned.m8n8k4.row.col.f64.f64.f64.f64 {%0, %1}, {%2}, {%3}, {%0, %1};"
               : "+d"(d[0]), "+d"(d[1])
               : "d"(a), "d"(b));
}

template <int TM>
__global__ void __launch_bounds__(256, 2) dgemm_kernel(int M, int N, int Kd, const double* __restrict__ A, long sa_m,
                                                    long sa_k, const double* __restrict__ B, long sb_k, long sb_n,
                                                    double* __restrict__ C, long sc_m, long sc_n, double alpha,
                                                    double beta, int flags) {
  constexpr int BM = 16 * TM;
  constexpr int MT = TM / 2;  // 8 x 8 tensor-core tiles per warp along M (four along N)
  // Two slices of each operand: the next one arrives while this one is used.  Element (k, x) sits at column
  // x ^ ((k & 3) << 2): a fragment load touches four k rows times four neighbouring columns per half warp, and the
  // swap of 4-column groups by k spreads them over all banks.
  __shared__ __align__(16) double As[2][kBK][BM];
  __shared__ __align__(16) double Bs[2][kBK][kBN];
  const int m0 = blockIdx.y * BM, n0 = blockIdx.x * kBN;
  if ((flags & kUpperOut) && m0 >= n0 + kBN) return;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int wm = (warp & 3) * (8 * MT), wn = (warp >> 2) * 32;  // the warp's corner inside the block's tile
  const int fr = lane >> 2, fk = lane & 3;                      // fragment row (or column) and k index of this lane
  const bool a_m_fast = (sa_m == 1), b_n_fast = (sb_n == 1);
  const int k_begin = (flags & kAUpper) ? m0 : 0;  // m0 is a multiple of 16
  const int k_end = (flags & kBUpper) ? min(Kd, n0 + kBN) : Kd;
  // One slice of both operands, global -> shared without passing through registers; elements outside the
  // operands are written as zeros (source size 0).
  auto fetch_slice = [&](int buf, int k0) {
#pragma unroll
    for (int i = 0; i < TM; ++i) {
      const int e = tid + i * 256;
      const int am = a_m_fast ? (e % BM) : (e >> 4), ak = a_m_fast ? (e / BM) : (e & 15);
      const bool in = (m0 + am < M && k0 + ak < Kd);
      async_copy8(&As[buf][ak][am ^ ((ak & 3) << 2)], in ? A + (long)(m0 + am) * sa_m + (long)(k0 + ak) * sa_k : A, in);
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int e = tid + i * 256;
      const int bn = b_n_fast ? (e & 63) : (e >> 4), bk = b_n_fast ? (e >> 6) : (e & 15);
      const bool in = (n0 + bn < N && k0 + bk < Kd);
      async_copy8(&Bs[buf][bk][bn ^ ((bk & 3) << 2)], in ? B + (long)(k0 + bk) * sb_k + (long)(n0 + bn) * sb_n : B, in);
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
  };
  double acc[MT][4][2] = {};
  if (k_begin < k_end) fetch_slice(0, k_begin);
  int buf = 0;
  for (int k0 = k_begin; k0 < k_end; k0 += kBK, buf ^= 1) {
    if (k0 + kBK < k_end) {
      fetch_slice(buf ^ 1, k0 + kBK);
      asm volatile("cp.async.wait_group 1;" ::: "memory");
    } else {
      asm volatile("cp.async.wait_group 0;" ::: "memory");
    }
    __syncthreads();
#pragma unroll
    for (int k = 0; k < kBK; k += 4) {
      // FP64 tensor-core step (8 x 8 x 4): this lane holds A[row fr][k fk] and B[k fk][column fr] of each tile
      double a[MT], b[4];
#pragma unroll
      for (int i = 0; i < MT; ++i) a[i] = As[buf][k + fk][(wm + 8 * i + fr) ^ (fk << 2)];
#pragma unroll
      for (int j = 0; j < 4; ++j) b[j] = Bs[buf][k + fk][(wn + 8 * j + fr) ^ (fk << 2)];
#pragma unroll
      for (int i = 0; i < MT; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) dmma_8x8x4(acc[i][j], a[i], b[j]);
    }
    __syncthreads();  // everyone is done with this slice before the next fetch overwrites it
  }
  // Accumulator layout: rows fr, columns 2 fk and 2 fk + 1 of each 8 x 8 tile.  Two passes over the outputs, all
  // loads of C before the first store: with run-time strides the compiler cannot tell that the addresses differ, and
  // a load placed after a store would wait for it, one memory round trip each.
  if (beta != 0.0) {
#pragma unroll
    for (int i = 0; i < MT; ++i)
#pragma unroll
      for (int j = 0; j < 4; ++j)
#pragma unroll
        for (int c = 0; c < 2; ++c) {
          const int m = m0 + wm + 8 * i + fr, n = n0 + wn + 8 * j + 2 * fk + c;
          const double v = (m < M && n < N) ? C[(long)m * sc_m + (long)n * sc_n] : 0.0;
          acc[i][j][c] = fma(alpha, acc[i][j][c], beta * v);
        }
  } else {
#pragma unroll
    for (int i = 0; i < MT; ++i)
#pragma unroll
      for (int j = 0; j < 4; ++j) acc[i][j][0] *= alpha, acc[i][j][1] *= alpha;
  }
#pragma unroll
  for (int i = 0; i < MT; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j)
#pragma unroll
      for (int c = 0; c < 2; ++c) {
        const int m = m0 + wm + 8 * i + fr, n = n0 + wn + 8 * j + 2 * fk + c;
        if (m < M && n < N) C[(long)m * sc_m + (long)n * sc_n] = acc[i][j][c];
      }
}

__global__ void bf16_to_f64_kernel(const uint16_t* __restrict__ in, double* __restrict__ out, long n) {
  const long i = (long)blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) out[i] = (double)__uint_as_float((uint32_t)in[i] << 16);
}

// Dead input channels (H_kk = 0) get H_kk = 1, and the mean of the diagonal after that fix goes to *mean_out.
// One block; the sum runs in a fixed order (thread-strided partial sums, then a tree), so it is deterministic.
__global__ void gptq_diag_mean_kernel(double* __restrict__ H, int K, unsigned char* __restrict__ dead,
                                      double* __restrict__ mean_out) {
  __shared__ double part[256];
  double s = 0.0;
  for (int k = threadIdx.x; k < K; k += 256) {
    double d = H[(long)k * K + k];
    const bool is_dead = (d == 0.0);
    if (is_dead) {
      d = 1.0;
      H[(long)k * K + k] = 1.0;
    }
    dead[k] = is_dead ? 1 : 0;
    s += d;
  }
  part[threadIdx.x] = s;
  __syncthreads();
  for (int w = 128; w > 0; w >>= 1) {
    if (threadIdx.x < w) part[threadIdx.x] += part[threadIdx.x + w];
    __syncthreads();
  }
  if (threadIdx.x == 0) *mean_out = part[0] / (double)K;
}

__global__ void gptq_damp_kernel(double* __restrict__ H, int K, const double* __restrict__ mean, double percdamp) {
  const int k = blockIdx.x * blockDim.x + threadIdx.x;
  if (k < K) H[(long)k * K + k] += percdamp * *mean;
}

// W = FP64(R) with the rows of dead input channels zeroed.
__global__ void gptq_init_w_kernel(const float* __restrict__ R, const unsigned char* __restrict__ dead,
                                   double* __restrict__ W, int K, int N) {
  const long i = (long)blockIdx.x * blockDim.x + threadIdx.x;
  if (i < (long)K * N) W[i] = dead[i / N] ? 0.0 : (double)R[i];
}

// ---------------------------------------------------------------------------------------------------------
// H = V V^T, V upper triangular, from the last block to the first (A holds H's upper triangle and ends as V).
// ---------------------------------------------------------------------------------------------------------

// The 64 x 64 diagonal block at j0, whose trailing updates are already applied: column 63 down to column 0, one
// barrier per column.  Sixteen threads share a row.  At column j every thread forms 1 / sqrt(pivot) itself, scales
// the entries of column j it needs on the fly (they stay unscaled in shared memory; the scaled column goes straight
// to global memory, nobody reads it again here) and updates its part of the columns to the left, so reads (column j)
// and writes (columns < j) of one step never meet.  A pivot that is not positive raises *not_pd.
constexpr int kDiagParts = 16;  // threads per row (4, 8 and 16 measure within 1 % of one another per layer)
constexpr int kDiagThreads = kDiagParts * kNb;
__global__ void __launch_bounds__(kDiagThreads) chol_diag_kernel(double* __restrict__ A, long ld, int j0, int* not_pd) {
  __shared__ double S[kNb][kNb + 1];
  const int t = threadIdx.x & (kNb - 1), part = threadIdx.x >> 6;
  for (int r = part; r < kNb; r += kDiagParts) S[r][t] = A[(long)(j0 + r) * ld + j0 + t];
  __syncthreads();
  for (int j = kNb - 1; j >= 0; --j) {
    const double d = S[j][j];
    const double inv = rsqrt(d), root = d * inv;  // one short chain per column instead of a root and a division
    if (threadIdx.x == j) {
      if (!(d > 0.0)) *not_pd = 1;
      A[(long)(j0 + j) * ld + j0 + j] = root;
    }
    if (t < j) {
      const double f = S[t][j] * inv;
      if (part == 0) A[(long)(j0 + t) * ld + j0 + j] = f;
      for (int c = t + part; c < j; c += kDiagParts) S[t][c] = fma(-f, S[c][j] * inv, S[t][c]);
    }
    __syncthreads();
  }
  // below the diagonal: zeros (the triangular inverse reads the whole block)
  for (int r = part; r < kNb; r += kDiagParts)
    if (t < r) A[(long)(j0 + r) * ld + j0 + t] = 0.0;
}

// The panel above the diagonal block: each row x of A[0:j0, j0:j0+64] becomes the solution of x D^T = row, D the
// factored diagonal block.  One thread per row, the row in registers.
__global__ void __launch_bounds__(kNb) chol_panel_kernel(double* __restrict__ A, long ld, int j0) {
  __shared__ double D[kNb][kNb + 1];
  __shared__ double rD[kNb];  // reciprocal diagonal: a product per column instead of a division in the serial chain
  const int t = threadIdx.x;
  for (int r = 0; r < kNb; ++r) D[r][t] = A[(long)(j0 + r) * ld + j0 + t];
  rD[t] = 1.0 / A[(long)(j0 + t) * ld + j0 + t];
  __syncthreads();
  const int row = blockIdx.x * kNb + t;
  if (row >= j0) return;
  double* p = A + (long)row * ld + j0;
  double b[kNb];
#pragma unroll
  for (int c = 0; c < kNb; ++c) b[c] = p[c];
#pragma unroll
  for (int c = kNb - 1; c >= 0; --c) {
    b[c] = b[c] * rD[c];
#pragma unroll
    for (int c2 = 0; c2 < c; ++c2) b[c2] = fma(-b[c], D[c2][c], b[c2]);
  }
#pragma unroll
  for (int c = 0; c < kNb; ++c) p[c] = b[c];
}

// ---------------------------------------------------------------------------------------------------------
// U = V^-1 (both upper triangular), block row by block row from the bottom.
// ---------------------------------------------------------------------------------------------------------

// Inverse of the 64 x 64 diagonal blocks of V from row `first` on (one block of threads each) into the same place of
// U: thread c solves D x = e_c.
__global__ void __launch_bounds__(kNb) triinv_diag_kernel(const double* __restrict__ V, double* __restrict__ U,
                                                          long ld, int first) {
  __shared__ double D[kNb][kNb + 1];
  const int t = threadIdx.x, i0 = first + blockIdx.x * kNb;
  for (int r = 0; r < kNb; ++r) D[r][t] = V[(long)(i0 + r) * ld + i0 + t];
  __syncthreads();
  double b[kNb];
#pragma unroll
  for (int r = 0; r < kNb; ++r) b[r] = (r == t) ? 1.0 : 0.0;
#pragma unroll
  for (int k = kNb - 1; k >= 0; --k) {
    b[k] = b[k] / D[k][k];
#pragma unroll
    for (int r = 0; r < k; ++r) b[r] = fma(-D[r][k], b[k], b[r]);
  }
#pragma unroll
  for (int r = 0; r < kNb; ++r) U[(long)(i0 + r) * ld + i0 + t] = b[r];
}

// ---------------------------------------------------------------------------------------------------------
// The sweep over one group of 64 input channels starting at k0 (Algorithm 1's inner loop).
// scale = FP32(max |w| / 7) over the group as it stands on entry; per channel code = clamp(round-half-even(w /
// scale), -8, 7) (0 for an all-zero group), err = (w - code * scale) / U_kk, later channels of the group -= err *
// U_kj.  Err [64, N] keeps the scaled errors for the update of the groups still to come.
// Two neighbouring lanes share an output channel: the even lane keeps the group's even input channels in registers,
// the odd lane the odd ones.  At step k both get w_k from its owner by a shuffle and compute code and error alike
// (same operations, same results), and each updates its own later channels: half the multiply-adds and half the
// unrolled code per thread.
// ---------------------------------------------------------------------------------------------------------
// MX: the same sweep on the MXFP4 grid of the MX variant (OCP MX v1.0): one E8M0 exponent per 32 input channels,
// floor(log2 max|w|) - 2 over the block as it stands when the sweep enters it, and E2M1 elements {0, 0.5, 1, 1.5, 2,
// 3, 4, 6} * 2^e, nearest with ties to the even code, saturating at 6, sign bit from the compensated weight.
constexpr int kGroupCols = 32;  // output channels per block of 64 threads
template <bool MX>
__global__ void __launch_bounds__(2 * kGroupCols) gptq_group_kernel(const double* __restrict__ W, int N,
                                                                    const double* __restrict__ U, long ldu, int k0,
                                                                    void* __restrict__ codes_out,
                                                                    void* __restrict__ scales_out,
                                                                    double* __restrict__ Err) {
  __shared__ double D[kNb][kNb + 1];
  __shared__ double rD[kNb];  // 1 / U_kk: the error is scaled by a product, which keeps one division out of the
                              // chain from one input channel to the next (the code is still decided by w / s)
  const int t = threadIdx.x;
  for (int r = 0; r < kNb; ++r) D[r][t] = U[(long)(k0 + r) * ldu + k0 + t];
  rD[t] = 1.0 / U[(long)(k0 + t) * ldu + k0 + t];
  __syncthreads();
  const int lane = t & 31, p = t & 1;
  const int col = blockIdx.x * kGroupCols + (t >> 1);
  const bool valid = col < N;           // both lanes of a pair agree; nobody leaves before the last shuffle
  const int n = valid ? col : N - 1;
  double w[kNb / 2];                    // input channels 2 i + p
#pragma unroll
  for (int i = 0; i < kNb / 2; ++i) w[i] = W[(long)(k0 + 2 * i + p) * N + n];
  double s = 0.0, inv_s = 0.0;          // INT4: the group's scale.  MX: 2^e of the running block and its reciprocal
  if constexpr (!MX) {
    double amax = 0.0;
#pragma unroll
    for (int i = 0; i < kNb / 2; ++i) amax = fmax(amax, fabs(w[i]));
    amax = fmax(amax, __shfl_xor_sync(0xffffffffu, amax, 1));
    const float s32 = (float)(amax / 7.0);  // FP64 quotient rounded once to FP32
    if (valid && p == 0) static_cast<float*>(scales_out)[(long)(k0 / kNb) * N + n] = s32;
    s = (double)s32;
  }
#pragma unroll
  for (int k = 0; k < kNb; ++k) {
    const int i = k >> 1;
    if constexpr (MX) {
      if ((k & 31) == 0) {  // entering a block of 32 input channels: its exponent from the weights as they stand
        double amax = 0.0;
#pragma unroll
        for (int i2 = 0; i2 < 16; ++i2) amax = fmax(amax, fabs(w[i + i2]));
        amax = fmax(amax, __shfl_xor_sync(0xffffffffu, amax, 1));
        int e = amax > 0.0 ? ilogb(amax) - 2 : -127;
        e = max(-127, min(125, e));
        s = scalbn(1.0, e);
        inv_s = scalbn(1.0, -e);
        if (valid && p == 0) static_cast<uint8_t*>(scales_out)[(long)((k0 + k) / 32) * N + n] = (uint8_t)(e + 127);
      }
    }
    const double wk = __shfl_sync(0xffffffffu, w[i], (lane & ~1) | (k & 1));
    double deq;
    int code;
    if constexpr (MX) {
      const double v = fmin(fabs(wk) * inv_s, 6.0);  // exact: the scale is a power of two
      // one comparison per midpoint between neighbouring magnitudes, strict where the lower neighbour is the even code
      const int idx = (v > 0.25) + (v >= 0.75) + (v > 1.25) + (v >= 1.75) + (v > 2.5) + (v >= 3.5) + (v > 5.0);
      const double mag = idx < 4 ? 0.5 * idx : (idx < 6 ? idx - 2.0 : 2.0 * idx - 8.0);
      deq = (wk < 0.0 ? -mag : mag) * s;
      code = idx + (wk < 0.0 ? 8 : 0);
    } else {
      double q = 0.0;
      if (s > 0.0) q = fmin(fmax(rint(wk / s), -8.0), 7.0);
      deq = q * s;
      code = (int)q;
    }
    const double e = (wk - deq) * rD[k];
    if (valid && p == (k & 1)) {
      if constexpr (MX) static_cast<uint8_t*>(codes_out)[(long)(k0 + k) * N + n] = (uint8_t)code;
      else static_cast<int8_t*>(codes_out)[(long)(k0 + k) * N + n] = (int8_t)code;
      Err[(long)k * N + n] = e;
    }
    if ((k & 1) == 0 && p == 1) w[i] -= e * D[k][k + 1];  // channel k + 1 lives in the odd lane
#pragma unroll
    for (int i2 = i + 1; i2 < kNb / 2; ++i2) w[i2] -= e * D[k][2 * i2 + p];
  }
}

// The temporaries of one call, carved out of one workspace (256-byte aligned pieces).
struct Workspace {
  double *H, *U, *Xd, *W, *Err, *T, *mean;
  unsigned char* dead;
  int* not_pd;
  size_t bytes;
  Workspace(unsigned char* base, int K, int N, int M_cal) {
    size_t off = 0;
    auto take = [&](size_t n) {
      unsigned char* p = reinterpret_cast<unsigned char*>(reinterpret_cast<uintptr_t>(base) + off);
      off += (n + 255) & ~static_cast<size_t>(255);
      return p;
    };
    const size_t kk = (size_t)K * K * sizeof(double);
    H = reinterpret_cast<double*>(take(kk));
    U = reinterpret_cast<double*>(take(kk));
    W = reinterpret_cast<double*>(take((size_t)K * N * sizeof(double)));
    Err = reinterpret_cast<double*>(take((size_t)2 * kLazy * N * sizeof(double)));  // two error batches
    T = reinterpret_cast<double*>(take((size_t)kBand * K * sizeof(double)));
    Xd = reinterpret_cast<double*>(take((size_t)M_cal * K * sizeof(double)));
    mean = reinterpret_cast<double*>(take(sizeof(double)));
    dead = take((size_t)K);
    not_pd = reinterpret_cast<int*>(take(sizeof(int)));
    bytes = off;
  }
};

// The second stream of a call and the two events that order it against the caller's stream.
struct SideStream {
  cudaStream_t stream = nullptr;
  cudaEvent_t ev_main = nullptr, ev_side = nullptr;
  bool create() {
    return cudaStreamCreateWithFlags(&stream, cudaStreamNonBlocking) == cudaSuccess &&
           cudaEventCreateWithFlags(&ev_main, cudaEventDisableTiming) == cudaSuccess &&
           cudaEventCreateWithFlags(&ev_side, cudaEventDisableTiming) == cudaSuccess;
  }
  ~SideStream() {
    if (ev_main) cudaEventDestroy(ev_main);
    if (ev_side) cudaEventDestroy(ev_side);
    if (stream) cudaStreamDestroy(stream);
  }
};

struct OwnedAllocation {
  void* p = nullptr;
  ~OwnedAllocation() { cudaFree(p); }
};

void dgemm(cudaStream_t st, int M, int N, int Kd, const double* A, long sa_m, long sa_k, const double* B, long sb_k,
           long sb_n, double* C, long sc_m, long sc_n, double alpha, double beta, int flags = 0) {
  if (M <= 0 || N <= 0) return;
  if (M > 64) {
    dim3 grid((N + kBN - 1) / kBN, (M + 127) / 128);
    dgemm_kernel<8><<<grid, 256, 0, st>>>(M, N, Kd, A, sa_m, sa_k, B, sb_k, sb_n, C, sc_m, sc_n, alpha, beta, flags);
  } else {
    dim3 grid((N + kBN - 1) / kBN, 1);
    dgemm_kernel<4><<<grid, 256, 0, st>>>(M, N, Kd, A, sa_m, sa_k, B, sb_k, sb_n, C, sc_m, sc_n, alpha, beta, flags);
  }
}


bool gptq_shape_ok(int K, int N, int M_cal) {
  return K > 0 && N > 0 && K % kNb == 0 && K <= 16384 && N <= 65536 && M_cal >= 0 && M_cal <= (1 << 20);
}

}  // namespace

extern "C" size_t w4a4_gptq_workspace_bytes(int K, int N, int M_cal) {
  if (!gptq_shape_ok(K, N, M_cal)) return 0;
  return Workspace(nullptr, K, N, M_cal).bytes;
}

namespace {

w4a4_status_t gptq_run(bool mx, int device, const float* R, const uint16_t* Xhat, int M_cal, const double* H_in, int K,
                       int N, double percdamp, void* codes, void* scales, void* workspace, size_t workspace_bytes,
                       void* stream) {
  if (R == nullptr || codes == nullptr || scales == nullptr) return W4A4_ERR_INVALID_ARG;
  if ((Xhat == nullptr) == (H_in == nullptr)) return W4A4_ERR_INVALID_ARG;  // exactly one source of H
  if (Xhat == nullptr) M_cal = 0;
  if (!gptq_shape_ok(K, N, M_cal)) return W4A4_ERR_SHAPE;
  if (Xhat != nullptr && M_cal <= 0) return W4A4_ERR_SHAPE;
  if (!(percdamp >= 0.0)) return W4A4_ERR_INVALID_ARG;
  const size_t need = Workspace(nullptr, K, N, M_cal).bytes;
  if (workspace != nullptr && (workspace_bytes < need || (reinterpret_cast<uintptr_t>(workspace) & 255) != 0))
    return W4A4_ERR_INVALID_ARG;
  if (cudaSetDevice(device) != cudaSuccess) return W4A4_ERR_CUDA;
  cudaDeviceProp prop;
  if (cudaGetDeviceProperties(&prop, device) != cudaSuccess) return W4A4_ERR_CUDA;
  if (prop.major != 10) return W4A4_ERR_ARCH;
  cudaStream_t st = static_cast<cudaStream_t>(stream);

  OwnedAllocation own;
  if (workspace == nullptr) {
    if (cudaMalloc(&own.p, need) != cudaSuccess) {
      cudaGetLastError();
      return W4A4_ERR_ALLOC;
    }
    workspace = own.p;
  }
  const Workspace d(static_cast<unsigned char*>(workspace), K, N, M_cal);
  SideStream side;
  if (!side.create()) {
    cudaGetLastError();
    return W4A4_ERR_CUDA;
  }
  const size_t kk = (size_t)K * K * sizeof(double);
  cudaMemsetAsync(d.not_pd, 0, sizeof(int), st);
  cudaMemsetAsync(d.U, 0, kk, st);

  // 1. H, its dead channels and damping.
  if (Xhat != nullptr) {
    const long n = (long)M_cal * K;
    bf16_to_f64_kernel<<<(unsigned)((n + 255) / 256), 256, 0, st>>>(Xhat, d.Xd, n);
    cudaMemsetAsync(d.H, 0, kk, st);
    dgemm(st, K, K, M_cal, d.Xd, 1, K, d.Xd, K, 1, d.H, K, 1, 1.0, 0.0, kUpperOut);
  } else {
    cudaMemcpyAsync(d.H, H_in, kk, cudaMemcpyDeviceToDevice, st);
  }
  gptq_diag_mean_kernel<<<1, 256, 0, st>>>(d.H, K, d.dead, d.mean);
  gptq_damp_kernel<<<(K + 255) / 256, 256, 0, st>>>(d.H, K, d.mean, percdamp);
  {
    const long n = (long)K * N;
    gptq_init_w_kernel<<<(unsigned)((n + 255) / 256), 256, 0, st>>>(R, d.dead, d.W, K, N);
  }

  // 2. H = V V^T in place (main stream) and U = V^-1 (side stream), band by band from the last channels.
  // Factorization: inside a band of kBand columns every 64-column block is factored, solved against all rows above
  // it and applied to the band's columns still to come; the columns to the left of the band then take the whole
  // band's panels in one product that is kBand deep.  Rows lo..hi of V are final once the band's blocks are done (the
  // product that follows only touches rows and columns below lo), so the side stream inverts that band meanwhile:
  // the diagonal part block by block (U[i, rest] = -inv(V_ii) (V[i, rest] U[rest, rest]), 64-row products), the
  // part to the right of it in two products that are kBand rows high.  The factorization's chain of small kernels
  // and the inverse's large products overlap.
  cudaEventRecord(side.ev_main, st);  // U is zeroed
  cudaStreamWaitEvent(side.stream, side.ev_main, 0);
  for (int hi = K; hi > 0;) {
    const int lo = hi - kBand > 0 ? hi - kBand : 0;
    for (int j0 = hi - kNb; j0 >= lo; j0 -= kNb) {
      chol_diag_kernel<<<1, kDiagThreads, 0, st>>>(d.H, K, j0, d.not_pd);
      if (j0 == 0) break;
      chol_panel_kernel<<<(j0 + kNb - 1) / kNb, kNb, 0, st>>>(d.H, K, j0);
      // H[0:j0, lo:j0] -= P P[lo:j0]^T, P = the panel just solved
      dgemm(st, j0, j0 - lo, kNb, d.H + j0, K, 1, d.H + (long)lo * K + j0, 1, K, d.H + lo, K, 1, -1.0, 1.0);
    }
    cudaEventRecord(side.ev_main, st);
    // H[0:lo, 0:lo] -= P P^T over the band's panels (upper triangle only)
    dgemm(st, lo, lo, hi - lo, d.H + lo, K, 1, d.H + lo, 1, K, d.H, K, 1, -1.0, 1.0, kUpperOut);

    cudaStream_t s2 = side.stream;
    cudaStreamWaitEvent(s2, side.ev_main, 0);
    triinv_diag_kernel<<<(hi - lo) / kNb, kNb, 0, s2>>>(d.H, d.U, K, lo);
    for (int i0 = hi - 2 * kNb; i0 >= lo; i0 -= kNb) {
      const int r0 = i0 + kNb, rest = hi - r0;
      dgemm(s2, kNb, rest, rest, d.H + (long)i0 * K + r0, K, 1, d.U + (long)r0 * K + r0, K, 1, d.T, K, 1, 1.0, 0.0,
            kBUpper);
      dgemm(s2, kNb, rest, kNb, d.U + (long)i0 * K + i0, K, 1, d.T, K, 1, d.U + (long)i0 * K + r0, K, 1, -1.0, 0.0);
    }
    const int band = hi - lo, right = K - hi;
    if (right > 0) {
      dgemm(s2, band, right, right, d.H + (long)lo * K + hi, K, 1, d.U + (long)hi * K + hi, K, 1, d.T, K, 1, 1.0, 0.0,
            kBUpper);
      dgemm(s2, band, right, band, d.U + (long)lo * K + lo, K, 1, d.T, K, 1, d.U + (long)lo * K + hi, K, 1, -1.0, 0.0,
            kAUpper);
    }
    hi = lo;
  }
  cudaEventRecord(side.ev_side, side.stream);
  cudaStreamWaitEvent(st, side.ev_side, 0);  // U is complete

  // 3. The sweep, group by group.  Inside a lazy batch of kLazy input channels each group's scaled errors update the
  // batch's groups still to come.  The channels after the batch take the whole batch in one product, W[later] -=
  // U[batch, later]^T Err, split in two: the next batch's channels on the main stream, the rest on the side stream
  // while the next batch is swept.  Both touch the same rows as the next batch's own products, so each main-stream
  // product first waits for the side stream's previous one; the error batches alternate between two buffers.
  int batch = 0;
  for (int b0 = 0; b0 < K; b0 += kLazy, ++batch) {
    const int b1 = b0 + kLazy < K ? b0 + kLazy : K;
    double* err_batch = d.Err + (long)(batch & 1) * kLazy * N;
    for (int k0 = b0; k0 < b1; k0 += kNb) {
      double* err = err_batch + (long)(k0 - b0) * N;
      const dim3 grid((N + kGroupCols - 1) / kGroupCols);
      if (mx) gptq_group_kernel<true><<<grid, 2 * kGroupCols, 0, st>>>(d.W, N, d.U, K, k0, codes, scales, err);
      else gptq_group_kernel<false><<<grid, 2 * kGroupCols, 0, st>>>(d.W, N, d.U, K, k0, codes, scales, err);
      const int r0 = k0 + kNb;
      dgemm(st, b1 - r0, N, kNb, d.U + (long)k0 * K + r0, 1, K, err, N, 1, d.W + (long)r0 * N, N, 1, -1.0, 1.0);
    }
    if (b1 == K) break;
    const int b2 = b1 + kLazy < K ? b1 + kLazy : K;  // end of the next batch
    cudaStreamWaitEvent(st, side.ev_side, 0);        // the side stream's product of the batch before
    dgemm(st, b2 - b1, N, b1 - b0, d.U + (long)b0 * K + b1, 1, K, err_batch, N, 1, d.W + (long)b1 * N, N, 1, -1.0, 1.0);
    cudaEventRecord(side.ev_main, st);
    cudaStreamWaitEvent(side.stream, side.ev_main, 0);
    dgemm(side.stream, K - b2, N, b1 - b0, d.U + (long)b0 * K + b2, 1, K, err_batch, N, 1, d.W + (long)b2 * N, N, 1,
          -1.0, 1.0);
    cudaEventRecord(side.ev_side, side.stream);
  }
  cudaStreamWaitEvent(st, side.ev_side, 0);

  int not_pd = 0;
  if (cudaMemcpyAsync(&not_pd, d.not_pd, sizeof(int), cudaMemcpyDeviceToHost, st) != cudaSuccess ||
      cudaStreamSynchronize(st) != cudaSuccess || cudaStreamSynchronize(side.stream) != cudaSuccess ||
      cudaGetLastError() != cudaSuccess)
    return W4A4_ERR_CUDA;
  return not_pd ? W4A4_ERR_INVALID_ARG : W4A4_OK;
}

}  // namespace

extern "C" w4a4_status_t w4a4_gptq_accumulate(int device, const uint16_t* Xhat, int M_cal, int K, double* H,
                                              void* stream) {
  if (Xhat == nullptr || H == nullptr) return W4A4_ERR_INVALID_ARG;
  if (!gptq_shape_ok(K, 1, M_cal) || M_cal <= 0) return W4A4_ERR_SHAPE;
  if (cudaSetDevice(device) != cudaSuccess) return W4A4_ERR_CUDA;
  cudaDeviceProp prop;
  if (cudaGetDeviceProperties(&prop, device) != cudaSuccess) return W4A4_ERR_CUDA;
  if (prop.major != 10) return W4A4_ERR_ARCH;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  constexpr int kChunkRows = 4096;  // tokens converted to FP64 at a time
  const int chunk = M_cal < kChunkRows ? M_cal : kChunkRows;
  OwnedAllocation xd;
  if (cudaMalloc(&xd.p, (size_t)chunk * K * sizeof(double)) != cudaSuccess) {
    cudaGetLastError();
    return W4A4_ERR_ALLOC;
  }
  double* Xd = static_cast<double*>(xd.p);
  for (int m0 = 0; m0 < M_cal; m0 += chunk) {
    const int rows = M_cal - m0 < chunk ? M_cal - m0 : chunk;
    const long n = (long)rows * K;
    bf16_to_f64_kernel<<<(unsigned)((n + 255) / 256), 256, 0, st>>>(Xhat + (size_t)m0 * K, Xd, n);
    dgemm(st, K, K, rows, Xd, 1, K, Xd, K, 1, H, K, 1, 1.0, 1.0, kUpperOut);
  }
  if (cudaStreamSynchronize(st) != cudaSuccess || cudaGetLastError() != cudaSuccess) return W4A4_ERR_CUDA;
  return W4A4_OK;
}

extern "C" w4a4_status_t w4a4_gptq_quantize(int device, const float* R, const uint16_t* Xhat, int M_cal,
                                            const double* H_in, int K, int N, double percdamp, int8_t* codes,
                                            float* scales, void* workspace, size_t workspace_bytes, void* stream) {
  return gptq_run(false, device, R, Xhat, M_cal, H_in, K, N, percdamp, codes, scales, workspace, workspace_bytes, stream);
}

extern "C" w4a4_status_t w4a4_mx_gptq_quantize(int device, const float* R, const uint16_t* Xhat, int M_cal,
                                               const double* H_in, int K, int N, double percdamp, uint8_t* codes,
                                               uint8_t* exps, void* workspace, size_t workspace_bytes, void* stream) {
  return gptq_run(true, device, R, Xhat, M_cal, H_in, K, N, percdamp, codes, exps, workspace, workspace_bytes, stream);
}
