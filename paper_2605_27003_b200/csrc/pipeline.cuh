// Pieces every tcgen05 GEMM of this library shares: tile constants, bounded mbarrier waits with their error
// codes, ring bookkeeping, the fused output activation, the parameter block and
// the weight expansion pre-pass.
//
// Every wait on an mbarrier is bounded: after WaitEnv::limit_ns without progress (or as soon as another CTA
// has reported an error) the role leaves its loop, the CTA records a code in *err and exits through the common
// tail that frees TMEM.  Nothing built on these helpers can spin forever.
#pragma once

#include <cuda_bf16.h>
#include <stdint.h>

#include "fp8_codes.cuh"
#include "ptx.cuh"

namespace w4a4 {

constexpr int kBM = 128;            // output tile rows (tokens) of one CTA
constexpr int kBN = 128;            // output tile columns (output channels)
constexpr int kBK = 128;            // K codes per pipeline stage = 2 quantization groups
constexpr int kGemmThreads = 640;
constexpr int kEpiWarp0 = 4, kEpiWarps = 16;
constexpr int kEpiCols = kBN / (kEpiWarps / 4);   // output channels per epilogue thread (32)

constexpr uint64_t kWaitLimitNs = 2000000000ull;     // 2 s: default limit of a bounded wait

enum GemmErr : int {
  kErrNone = 0,
  kErrProducerWait = 101,
  kErrMmaWait = 103,
  kErrEpilogueWait = 104,
  kErrProbeWait = 105,
};

struct WaitEnv {
  int* g_err;                // device-global error word (0 = healthy)
  volatile int* s_abort;     // CTA-local abort flag in shared memory
  uint64_t limit_ns;         // how long a wait may go without progress
};

// Slow path of a bounded wait, kept out of line so that the callers' loops stay small.  ROLE only separates the
// instantiations: an out-of-line function called from warp roles that run under different register budgets
// (setmaxnreg) would have to fit all of them.
template <int BACKOFF_NS, int ROLE>
__device__ __noinline__ bool bounded_wait_slow(uint32_t bar, uint32_t parity, int* g_err, volatile int* s_abort,
                                               uint64_t limit_ns, int code) {
  const uint64_t t0 = global_timer_ns();
  uint32_t spins = 0;
  for (;;) {
    if (mbar_try_wait(bar, parity)) return true;
    if (BACKOFF_NS > 0) __nanosleep(BACKOFF_NS);  // roles that run ahead poll lazily: issue slots belong to the epilogue
    if ((++spins & 31u) == 0) {
      if (*s_abort) return false;
      if (*reinterpret_cast<volatile int*>(g_err) != 0) {
        *s_abort = 1;
        return false;
      }
      if (global_timer_ns() - t0 > limit_ns) {
        atomicCAS(g_err, 0, code);
        *s_abort = 1;
        return false;
      }
    }
  }
}

// Bounded wait.  Returns false if the CTA should give up.  mbarrier.try_wait itself blocks for a while before it
// reports failure, so a short inline run of attempts covers every hand-over of a healthy pipeline; only a wait that
// outlasts it pays for the out-of-line call and its timer reads.
template <int BACKOFF_NS = 0, int ROLE = 0>
__device__ __forceinline__ bool bounded_wait(uint32_t bar, uint32_t parity, const WaitEnv& env, int code) {
#pragma unroll 1
  for (int i = 0; i < 16; ++i) {
    if (mbar_try_wait(bar, parity)) return true;
  }
  return bounded_wait_slow<BACKOFF_NS, ROLE>(bar, parity, env.g_err, env.s_abort, env.limit_ns, code);
}

// One lane of a converged warp.
__device__ __forceinline__ bool elect_one_lane() {
  uint32_t pred;
  asm volatile(
      "{\n"
      ".reg .pred p;\n"
      "elect.sync _|p, 0xffffffff;\n"
      "selp.u32 %0, 1, 0, p;\n"
      "}\n"
      : "=r"(pred));
  return pred != 0;
}

// Position in a ring of N mbarrier pairs: slot index and the parity of the phase a consumer waits
// for (a producer waits for parity ^ 1).  Advanced incrementally: no division in the hot loops.
template <int N>
struct Ring {
  uint32_t slot = 0, parity = 0;
  __device__ __forceinline__ void advance() {
    if (++slot == N) {
      slot = 0;
      parity ^= 1u;
    }
  }
};

// Output activation of the layer (W4A4_ACT_*), applied in FP32 before the BF16 rounding.
// GELU, tanh form: 0.5 y (1 + tanh u) with u = sqrt(2/pi) (y + 0.044715 y^3) equals y * sigmoid(2 u) =
// y / (1 + exp(-2 u)); written that way it needs one ex2 and one reciprocal (both accurate to about 2^-22) instead
// of a full-precision tanh, and has no cancellation for negative y.
__device__ __forceinline__ float apply_activation(float y, int act) {
  if (act == 1) {
    const float y2 = y * y;
    // -2 u log2(e) = y (c1 + c3 y^2)
    const float t = y * fmaf(y2, -2.0f * 0.7978845608028654f * 0.044715f * 1.4426950408889634f,
                             -2.0f * 0.7978845608028654f * 1.4426950408889634f);
    float e;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(e) : "f"(t));
    float rcp;
    asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(rcp) : "f"(1.0f + e));
    return y * rcp;
  }
  return y;
}

struct GemmParams {
  const float* bias;    // [N] or nullptr
  uint16_t* Y;          // [M, N] BF16
  int M, N, K, r;
  int tiles_m, tiles_n;
  int sc_tiles;         // column tiles per super-column of the tile order (tiles_n: plain row-major order)
  int* err;
  uint64_t wait_limit_ns;
  int32_t* dbg_P;       // debug tap: [kBM, G, kBN] or nullptr
  int dbg_m0, dbg_n0;
  int dbg_stall_stage;  // test hook of the tap instantiation: every CTA's producer skips its stage of this number (-1: none)
  // Clip-ratio search (Eq. 10): when yref is set, Y is not stored; the squared distance between the layer's
  // BF16 output and yref is accumulated into *sq_err instead.
  const uint16_t* yref; // [M, N] BF16 or nullptr
  double* sq_err;
  int act;              // output activation: 0 none, 1 GELU (tanh form)
};

// Weight codes at rest -> the E4M3 byte image kernel 2 reads: [N, K/2] packed as code + 8 (byte j of a row holds
// K offsets 2 j in its low nibble and 2 j + 1 in its high nibble) -> [N, K] bytes.  One thread turns 32 codes
// (16 bytes in) into 32 bytes out; each half-word of an input word is one byte-permute selector.
__global__ void expand_weight_kernel(const uint4* __restrict__ packed, uint4* __restrict__ out, size_t chunks) {
  const size_t i = static_cast<size_t>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (i >= chunks) return;
  const uint4 w = __ldg(packed + i);
  out[2 * i] = make_uint4(e4m3_of_offset_nibbles4(w.x), e4m3_of_offset_nibbles4(w.x >> 16), e4m3_of_offset_nibbles4(w.y),
                          e4m3_of_offset_nibbles4(w.y >> 16));
  out[2 * i + 1] = make_uint4(e4m3_of_offset_nibbles4(w.z), e4m3_of_offset_nibbles4(w.z >> 16),
                              e4m3_of_offset_nibbles4(w.w), e4m3_of_offset_nibbles4(w.w >> 16));
}

// The end every GEMM kernel of this library shares after its role loops: if a wait gave up, copies that may
// still be in flight get time to land before the CTA's shared memory is released.
__device__ __forceinline__ void drain_after_abort(volatile int* s_abort) {
  if (*s_abort) {
    const uint64_t t0 = global_timer_ns();
    while (global_timer_ns() - t0 < 200000ull) __nanosleep(1000);
    __syncthreads();
  }
}

// Exercises the give-up path of bounded_wait without any pipeline around it: one warp waits for a phase of an
// mbarrier that nobody ever completes.  No copy, tensor-core operation or TMEM allocation is involved, so there is
// nothing to drain: after limit_ns the wait records kErrProbeWait in *err and the kernel returns normally.
__global__ void wait_probe_kernel(int* err, uint64_t limit_ns) {
  __shared__ __align__(8) uint64_t bar;
  __shared__ int s_abort;
  if (threadIdx.x == 0) {
    s_abort = 0;
    mbar_init(smem_u32(&bar), 1);
    mbar_fence_init();
  }
  __syncthreads();
  const WaitEnv env{err, &s_abort, limit_ns};
  bounded_wait<0, 9>(smem_u32(&bar), 0, env, kErrProbeWait);
}

}  // namespace w4a4
