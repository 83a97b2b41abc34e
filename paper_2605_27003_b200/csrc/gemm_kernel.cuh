// Kernel 2: fused W4A4 GEMM + per-group rescale + low-rank up-projection + bias + BF16 store.
//
//   Eq. 7 / 11    Y[m,n] = sum_g  P[m,g,n] * s[m,g] * sw[g,n]  +  sum_j T[m,j] L2[j,n]  +  b[n]
//                 P[m,g,n] = sum_{k in group g} q[m,k] qw[k,n]            (exact: integers in FP32)
//
// The 4-bit codes go through the tensor core as E4M3 bytes (fp8_codes.cuh): tcgen05.mma kind::f8f6f4 runs
// at the 8-bit rate and leaves every group's partial sums in TMEM as exact integers already in FP32, so
// the epilogue needs no int -> float conversion.
//
// Persistent kernel: one CTA per SM walks over 128 x 128 output tiles (column tile fastest, so the
// CTAs running at any moment share a few row blocks of A and all of B through L2).  Both operands arrive
// as E4M3 bytes: the activation codes straight from kernel 1, the weight codes from expand_weight_kernel,
// which runs right before this kernel and turns the layer's nibble-packed weights (their format at rest)
// into an N x K byte image that stays in L2 for the duration of the GEMM.  Nothing is unpacked on the SM:
// its issue slots and shared-memory port belong to the epilogue.  Every role loops with all 32 lanes of its warp
// (waits are voted, only the TMA / tcgen05 instructions are predicated on one elected lane), which keeps ring
// positions, addresses and descriptors warp-uniform for the compiler.  Warp roles:
//   warp 0        producer: per stage (128 K-codes = two quantization groups) one TMA for the
//                 128 x 128-byte A tile and one for the B tile, both with the 128-byte swizzle the tensor
//                 core expects, into a slot of the operand ring, plus the matching 2 x 128 blocks of weight
//                 scales and of activation scales into the "scale" ring (same mbarrier; that ring is deep
//                 enough to need no barriers of its own).  The BF16 low-rank operands T and L2 use the
//                 same ring.
//   warp 1        MMA issuer: per stage four tcgen05.mma kind::f8f6f4 (K=32 each), two per group,
//                 each group into its own 128-column half of a 256-column TMEM slot (2 slots), so that
//                 every group's partial sums stay separate; kind::f16 for the low-rank product
//                 (first slot of a tile).  One barrier round trip per stage, not per group.
//   warp 2        TMEM allocation / release.
//   warps 4-19    epilogue: TMEM -> registers with the 32x32b shape (a thread reads its own TMEM lane, i.e. one
//                 token row; by far the fastest of the load shapes: ~830 B/clk/SM against ~250 for the
//                 16x256b accumulator-fragment shape), * sw[g,n] * s[m,g] into 32 FP32 accumulators per thread
//                 (one row x 32 output channels), finally + bias, BF16.  Sixteen warps, four per scheduler,
//                 so that TMEM and shared-memory latencies of one warp hide behind the arithmetic of others.
//
// The epilogue's FP32 work (one multiply and one fused multiply-add per partial sum, all with distinct
// register operands) and the shared-memory port (operand tiles written by TMA and read by the tensor core,
// plus the broadcast loads of the weight scales) are what bound this kernel, not the tensor core; the
// epilogue loop is therefore written one stage (two groups) per iteration with all ring bookkeeping kept
// incremental.
//
// Every wait on an mbarrier is bounded: after kWaitLimitNs without progress (or as soon as another
// CTA has reported an error) the role leaves its loop, the CTA records a code in *err and exits
// through the common tail that frees TMEM.  Nothing in this file can spin forever.
#pragma once

#include <cuda_bf16.h>
#include <stdint.h>

#include "fp8_codes.cuh"
#include "ptx.cuh"

namespace w4a4 {

constexpr int kBM = 128;            // output tile rows (tokens)
constexpr int kBN = 128;            // output tile columns (output channels)
constexpr int kBK = 128;            // K codes per pipeline stage = 2 quantization groups
constexpr int kOpStages = 6;        // operand ring: A and B tiles of one stage, one byte per code, tensor-core ready
constexpr int kScaleStages = 12;   // ring of scale blocks (2 groups x (kBN weight scales + kBM activation scales));
                                   // deeper than the TMA producer can ever run ahead of the epilogue, so it needs no barriers
constexpr int kTmemSlots = 2;       // TMEM slots of 2 x kBN columns: one per stage in flight
constexpr int kGemmThreads = 640;
constexpr int kEpiWarp0 = 4, kEpiWarps = 16;
constexpr int kEpiCols = kBN / (kEpiWarps / 4);   // output channels per epilogue thread (32)
constexpr int kRegsControl = 40, kRegsEpilogue = 104;   // setmaxnreg budgets per role: 4 x 32 x 40 + 16 x 32 x 104 fits the
                                                        // 640 x 96 registers the CTA is launched with
// setmaxnreg.inc blocks until the CTA's own allocation (threads x the compiled register count, which the launch
// bound fixes at 96) has that many registers free: a budget above it never returns.
static_assert(kEpiWarp0 * 32 * kRegsControl + kEpiWarps * 32 * kRegsEpilogue <= kGemmThreads * 96,
              "setmaxnreg budgets exceed the registers the CTA is launched with");

constexpr uint32_t kOpATile = kBM * kBK;             // 16 KiB
constexpr uint32_t kOpBTile = kBN * kBK;             // 16 KiB
constexpr uint32_t kOpStageBytes = kOpATile + kOpBTile;
constexpr uint32_t kScaleStageBytes = 2 * (kBN + kBM) * 4;   // 2 KiB: sw[2][kBN] then sa[2][kBM]
constexpr uint32_t kNumBarriers = 2 * kOpStages + 2 * kTmemSlots;
constexpr uint32_t kGemmSmemBytes = 1024 /*alignment slack*/ + kOpStages * kOpStageBytes +
                                    kScaleStages * kScaleStageBytes + kNumBarriers * 8 + 16;

constexpr uint64_t kWaitLimitNs = 2000000000ull;     // 2 s

enum GemmErr : int {
  kErrNone = 0,
  kErrProducerWait = 101,
  kErrMmaWait = 103,
  kErrEpilogueWait = 104,
};

struct WaitEnv {
  int* g_err;                // device-global error word (0 = healthy)
  volatile int* s_abort;     // CTA-local abort flag in shared memory
};

// Slow path of a bounded wait, kept out of line so that the callers' loops stay small.
template <int BACKOFF_NS>
__device__ __noinline__ bool bounded_wait_slow(uint32_t bar, uint32_t parity, int* g_err, volatile int* s_abort,
                                               int code) {
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
      if (global_timer_ns() - t0 > kWaitLimitNs) {
        atomicCAS(g_err, 0, code);
        *s_abort = 1;
        return false;
      }
    }
  }
}

// Bounded wait.  Returns false if the CTA should give up.
template <int BACKOFF_NS = 0>
__device__ __forceinline__ bool bounded_wait(uint32_t bar, uint32_t parity, const WaitEnv& env, int code) {
  if (mbar_try_wait(bar, parity)) return true;
  return bounded_wait_slow<BACKOFF_NS>(bar, parity, env.g_err, env.s_abort, code);
}

// Position in a ring of N mbarrier pairs: slot index and the parity of the phase a consumer waits
// for (a producer waits for parity ^ 1).  Advanced incrementally: no division in the hot loops.
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

template <int N>
__device__ __forceinline__ void set_max_regs_inc() {
  asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(N));
}
template <int N>
__device__ __forceinline__ void set_max_regs_dec() {
  asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(N));
}

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
  int* err;
  int32_t* dbg_P;       // debug tap: [kBM, G, kBN] or nullptr
  int dbg_m0, dbg_n0;
  // Clip-ratio search (Eq. 10): when yref is set, Y is not stored; the squared distance between the layer's
  // BF16 output and yref is accumulated into *sq_err instead.
  const uint16_t* yref; // [M, N] BF16 or nullptr
  double* sq_err;
  int act;              // output activation: 0 none, 1 GELU (tanh form)
};

// Rescales one fragment (32 token rows x 16 columns: one row x 16 channels per thread) of a group's partial
// sums P (integers held in FP32) into the FP32 accumulators:  acc += P * sw[channel] * sa[row].
//   v     the fragment as loaded by tmem_ld_32x32b_x16: v[c] is column c of the thread's row
//   swp   the 16 weight scales of those columns in shared memory (the same for every lane: broadcast loads)
//   sa    activation scale of the thread's row
//   acc   8 accumulator pairs, pair k = columns 2 k, 2 k + 1
template <bool DEBUG>
__device__ __forceinline__ void rescale_fragment(const uint32_t (&v)[16], const float4* swp, float sa, float2* acc,
                                                 int32_t* dbg_row) {
  const float2 s2 = make_float2(sa, sa);
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const float4 w = swp[i];
    const float2 p0 = make_float2(__uint_as_float(v[4 * i]), __uint_as_float(v[4 * i + 1]));
    const float2 p1 = make_float2(__uint_as_float(v[4 * i + 2]), __uint_as_float(v[4 * i + 3]));
    acc[2 * i] = __ffma2_rn(__fmul2_rn(p0, make_float2(w.x, w.y)), s2, acc[2 * i]);
    acc[2 * i + 1] = __ffma2_rn(__fmul2_rn(p1, make_float2(w.z, w.w)), s2, acc[2 * i + 1]);
    if (DEBUG) {
      if (dbg_row != nullptr) {
        dbg_row[4 * i] = static_cast<int32_t>(p0.x);
        dbg_row[4 * i + 1] = static_cast<int32_t>(p0.y);
        dbg_row[4 * i + 2] = static_cast<int32_t>(p1.x);
        dbg_row[4 * i + 3] = static_cast<int32_t>(p1.y);
      }
    }
  }
}

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

template <bool DEBUG>
__global__ void __launch_bounds__(kGemmThreads, 1)
gemm_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
            const __grid_constant__ CUtensorMap tmSW, const __grid_constant__ CUtensorMap tmSA,
            const __grid_constant__ CUtensorMap tmT,
            const __grid_constant__ CUtensorMap tmL2, const GemmParams p) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* smem = smem_raw + (smem_base - smem_u32(smem_raw));
  const uint32_t op_base = smem_base;
  const uint32_t scale_base = op_base + kOpStages * kOpStageBytes;
  const uint32_t bar_base = scale_base + kScaleStages * kScaleStageBytes;
  const uint32_t bar_op_full = bar_base;
  const uint32_t bar_op_empty = bar_op_full + 8 * kOpStages;
  const uint32_t bar_tmem_full = bar_op_empty + 8 * kOpStages;
  const uint32_t bar_tmem_empty = bar_tmem_full + 8 * kTmemSlots;
  const uint32_t misc_off = (bar_tmem_empty + 8 * kTmemSlots) - smem_base;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + misc_off);
  volatile int* s_abort = reinterpret_cast<volatile int*>(smem + misc_off + 4);

  const int warp = __shfl_sync(0xffffffffu, static_cast<int>(threadIdx.x >> 5), 0), lane = threadIdx.x & 31;  // provably warp-uniform
  const int G = p.K >> 6;
  const int n_int_stages = (G + 1) >> 1;
  const int n_lr_stages = p.r > 0 ? (2 * p.r + 63) / 64 : 0;
  const int num_tiles = p.tiles_m * p.tiles_n;
  const WaitEnv env{p.err, s_abort};

  if (threadIdx.x == 0) {
    *s_abort = (*reinterpret_cast<volatile int*>(p.err) != 0) ? 1 : 0;
    for (int i = 0; i < kOpStages; ++i) {
      mbar_init(bar_op_full + 8 * i, 1);
      mbar_init(bar_op_empty + 8 * i, 1);
    }
    for (int i = 0; i < kTmemSlots; ++i) {
      mbar_init(bar_tmem_full + 8 * i, 1);
      mbar_init(bar_tmem_empty + 8 * i, kEpiWarps);
    }
    mbar_fence_init();
    fence_proxy_async_smem();
    tma_prefetch_desc(&tmA);
    tma_prefetch_desc(&tmB);
    tma_prefetch_desc(&tmSW);
    tma_prefetch_desc(&tmSA);
    if (p.r > 0) {
      tma_prefetch_desc(&tmT);
      tma_prefetch_desc(&tmL2);
    }
  }
  if (warp == 2) {
    tmem_alloc(smem_u32(tmem_slot), 512);
    tmem_relinquish();
    tc_fence_before_sync();
  }
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = __shfl_sync(0xffffffffu, *tmem_slot, 0);
  const bool live = __all_sync(0xffffffffu, *s_abort == 0);

  // Per tile the TMEM slots are used by: [one slot for the low-rank product, if r > 0] followed by
  // one slot per K stage (two groups, 128 columns each).
  if (warp < kEpiWarp0) {
    set_max_regs_dec<kRegsControl>();
    if (live && warp == 0) {
      // ------------------------------------------------------------------ TMA producer
      // All lanes run the loop (waits included) and one elected lane issues: what the TMA and tcgen05
      // instructions take as operands then stays warp-uniform for the compiler, which keeps it in uniform
      // registers instead of converting per instruction.
      const bool issuer = elect_one_lane();
      // Slots of the operand ring in the order the MMA warp consumes them: per tile the low-rank stages
      // (T and the duplicated L2 factor, BF16) first, then the code stages with their scales.
      Ring<kOpStages> op;
      Ring<kScaleStages> sc;
      bool ok = true;
      for (int tile = blockIdx.x; ok && tile < num_tiles; tile += gridDim.x) {
        const int m0 = (tile / p.tiles_n) * kBM, n0 = (tile % p.tiles_n) * kBN;
        for (int st = 0; st < n_lr_stages + n_int_stages; ++st) {
          ok = __all_sync(0xffffffffu, bounded_wait<128>(bar_op_empty + 8 * op.slot, op.parity ^ 1u, env, kErrProducerWait));
          if (!ok) break;
          const uint32_t full = bar_op_full + 8 * op.slot;
          const uint32_t dst = op_base + op.slot * kOpStageBytes;
          if (st < n_lr_stages) {
            if (issuer) {
              mbar_arrive_expect_tx(full, kOpStageBytes);
              tma_load_2d(dst, &tmT, full, st * 64, m0);
              tma_load_2d(dst + kOpATile, &tmL2, full, st * 64, n0);
            }
          } else {
            const int ks = st - n_lr_stages;
            const uint32_t sdst = scale_base + sc.slot * kScaleStageBytes;
            if (issuer) {
              mbar_arrive_expect_tx(full, kOpStageBytes + kScaleStageBytes);
              tma_load_2d(dst, &tmA, full, ks * kBK, m0);
              tma_load_2d(dst + kOpATile, &tmB, full, ks * kBK, n0);
              tma_load_2d(sdst, &tmSW, full, n0, 2 * ks);
              tma_load_2d(sdst + 2 * kBN * 4, &tmSA, full, m0, 2 * ks);
            }
            sc.advance();
          }
          op.advance();
        }
      }
    } else if (live && warp == 1) {
      // ------------------------------------------------------------------ MMA issuer (all lanes loop, one issues)
      constexpr uint32_t idesc_f8 = umma_idesc(1, 0, kBM, kBN);
      constexpr uint32_t idesc_bf16 = umma_idesc(1, 1, kBM, kBN);
      const bool issuer = elect_one_lane();
      Ring<kOpStages> op;
      Ring<kTmemSlots> tm;
      bool ok = true;
      for (int tile = blockIdx.x; ok && tile < num_tiles; tile += gridDim.x) {
        if (n_lr_stages > 0) {
          ok = __all_sync(0xffffffffu, bounded_wait<64>(bar_tmem_empty + 8 * tm.slot, tm.parity ^ 1u, env, kErrMmaWait));
          for (int l = 0; ok && l < n_lr_stages; ++l) {
            ok = __all_sync(0xffffffffu, bounded_wait<64>(bar_op_full + 8 * op.slot, op.parity, env, kErrMmaWait));
            if (!ok) break;
            tc_fence_after_sync();
            const uint32_t a = op_base + op.slot * kOpStageBytes, b = a + kOpATile;
            if (issuer) {
#pragma unroll
              for (int kk = 0; kk < 4; ++kk) {
                umma_f16(tmem_base + tm.slot * 2 * kBN, umma_desc_k_sw128(a, 32 * kk), umma_desc_k_sw128(b, 32 * kk),
                         idesc_bf16, (l > 0 || kk > 0) ? 1u : 0u);
              }
              umma_commit(bar_op_empty + 8 * op.slot);
            }
            op.advance();
          }
          if (!ok) break;
          if (issuer) umma_commit(bar_tmem_full + 8 * tm.slot);
          tm.advance();
        }
        for (int st = 0; ok && st < n_int_stages; ++st) {
          ok = __all_sync(0xffffffffu, bounded_wait<64>(bar_tmem_empty + 8 * tm.slot, tm.parity ^ 1u, env, kErrMmaWait) &&
                                           bounded_wait<64>(bar_op_full + 8 * op.slot, op.parity, env, kErrMmaWait));
          if (!ok) break;
          tc_fence_after_sync();
          const uint32_t a = op_base + op.slot * kOpStageBytes, b = a + kOpATile;
          const uint32_t d = tmem_base + tm.slot * 2 * kBN;
          const int groups = (2 * st + 1 < G) ? 2 : 1;
          if (issuer) {
#pragma unroll
            for (int kk = 0; kk < 4; ++kk) {  // bytes [32 kk, 32 kk + 32) of every row: group kk / 2, K half kk % 2
              if (kk < 2 * groups) {
                umma_f8(d + (kk >> 1) * kBN, umma_desc_k_sw128(a, 32 * kk), umma_desc_k_sw128(b, 32 * kk), idesc_f8,
                        kk & 1);
              }
            }
            umma_commit(bar_op_empty + 8 * op.slot);
            umma_commit(bar_tmem_full + 8 * tm.slot);
          }
          op.advance();
          tm.advance();
        }
      }
    }
  } else {
    set_max_regs_inc<kRegsEpilogue>();
    if (live) {
      // ------------------------------------------------------------------ epilogue warps
      // Warp ew owns TMEM lanes 32 * (ew % 4) .. +31 (token rows) and the 32-column block ew / 4; a thread owns
      // one row (its lane) and the block's 32 output channels.  Four epilogue warps per scheduler hide one
      // another's TMEM and shared-memory latencies.  Software pipeline over fragments of 16 columns: while one
      // fragment is being rescaled the next TMEM load (and, at stage boundaries, the barrier wait in front of
      // it) is already in flight.
      const int ew = warp - kEpiWarp0;
      const int quarter = ew & 3, colblk = ew >> 2;
      const uint32_t t_lane = tmem_base + (static_cast<uint32_t>(32 * quarter) << 16) + kEpiCols * colblk;
      // Per scale stage: sw[2][kBN] then sa[2][kBM] floats.  The warp's weight scales start at float
      // kEpiCols colblk, the thread's activation scale is float 2 kBN + 32 quarter + lane.
      const float* sw_warp = reinterpret_cast<const float*>(smem + (scale_base - smem_base)) + kEpiCols * colblk;
      const float* sa_thread = reinterpret_cast<const float*>(smem + (scale_base - smem_base)) + 2 * kBN + 32 * quarter + lane;
      Ring<kTmemSlots> tm;
      Ring<kScaleStages> sc;
      bool ok = true;
      for (int tile = blockIdx.x; ok && tile < num_tiles; tile += gridDim.x) {
        const int m0 = (tile / p.tiles_n) * kBM, n0 = (tile % p.tiles_n) * kBN;
        const int row = m0 + 32 * quarter + lane;
        const int ch0 = n0 + kEpiCols * colblk;
        const bool dbg_tile = DEBUG && p.dbg_P != nullptr && m0 == p.dbg_m0 && n0 == p.dbg_n0;
        float2 acc[16];  // pair k: channels ch0 + 2 k, ch0 + 2 k + 1
        uint32_t vA[16], vB[16];
        // First slot of the tile.
        ok = __all_sync(0xffffffffu, bounded_wait(bar_tmem_full + 8 * tm.slot, tm.parity, env, kErrEpilogueWait));
        if (!ok) break;
        tc_fence_after_sync();
        tmem_ld_32x32b_x16(t_lane + tm.slot * 2 * kBN, vA);
        tmem_wait_ld();
        if (n_lr_stages > 0) {
          // The low-rank product T L2 (FP32) seeds the accumulators.
          tmem_ld_32x32b_x16(t_lane + 16 + tm.slot * 2 * kBN, vB);
#pragma unroll
          for (int k = 0; k < 8; ++k) acc[k] = make_float2(__uint_as_float(vA[2 * k]), __uint_as_float(vA[2 * k + 1]));
          tmem_wait_ld();
          tc_fence_before_sync();
          __syncwarp();
          if (lane == 0) mbar_arrive(bar_tmem_empty + 8 * tm.slot);
          tm.advance();
          ok = __all_sync(0xffffffffu, bounded_wait(bar_tmem_full + 8 * tm.slot, tm.parity, env, kErrEpilogueWait));
          if (!ok) break;
          tc_fence_after_sync();
          tmem_ld_32x32b_x16(t_lane + tm.slot * 2 * kBN, vA);
#pragma unroll
          for (int k = 0; k < 8; ++k) acc[8 + k] = make_float2(__uint_as_float(vB[2 * k]), __uint_as_float(vB[2 * k + 1]));
          tmem_wait_ld();
        } else {
#pragma unroll
          for (int j = 0; j < 16; ++j) acc[j] = make_float2(0.0f, 0.0f);
        }
        // Invariant at the top of each iteration: the stage's TMEM slot has been waited for and vA
        // holds the first 16-column fragment of its first group.
        float2 (&acc_lo)[8] = *reinterpret_cast<float2(*)[8]>(&acc[0]);  // channels ch0 .. ch0 + 15
        float2 (&acc_hi)[8] = *reinterpret_cast<float2(*)[8]>(&acc[8]);  // channels ch0 + 16 .. ch0 + 31
        for (int st = 0; st < n_int_stages; ++st) {
          const int g0 = 2 * st;
          const bool two = g0 + 1 < G;
          const bool last_stage = st + 1 == n_int_stages;
          const uint32_t t_grp = t_lane + tm.slot * 2 * kBN;
          tmem_ld_32x32b_x16_before(t_grp + 16, vB, vA[0]);
          // The stage's scales landed before the MMA that produced this slot was even issued (they ride
          // on the operand tiles' mbarrier), so they can be read without a wait of their own.
          const float4* swp = reinterpret_cast<const float4*>(sw_warp + sc.slot * (kScaleStageBytes / 4));
          const float* sap = sa_thread + sc.slot * (kScaleStageBytes / 4);
          const float sa0 = sap[0], sa1 = sap[kBM];  // first / second group of the stage
          int32_t* d0 = nullptr;
          if (DEBUG) {
            if (dbg_tile) d0 = p.dbg_P + (static_cast<size_t>(32 * quarter + lane) * G + g0) * kBN + kEpiCols * colblk;
          }
          // ---- group g0
          rescale_fragment<DEBUG>(vA, swp, sa0, acc, d0);
          tmem_wait_ld_after(acc_lo);
          if (two) {
            tmem_ld_32x32b_x16_before(t_grp + kBN, vA, vB[0]);
          } else {
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_tmem_empty + 8 * tm.slot);
          }
          rescale_fragment<DEBUG>(vB, swp + 4, sa0, acc + 8, DEBUG && d0 ? d0 + 16 : nullptr);
          if (two) {
            // ---- group g0 + 1
            tmem_wait_ld_after(acc_hi);
            tmem_ld_32x32b_x16_before(t_grp + kBN + 16, vB, vA[0]);
            if (DEBUG) {
              if (dbg_tile) d0 += kBN;
            }
            rescale_fragment<DEBUG>(vA, swp + kBN / 4, sa1, acc, d0);
            tmem_wait_ld_after(acc_lo);
            // The whole slot is in registers: hand it back to the MMA warp.
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_tmem_empty + 8 * tm.slot);
          }
          tm.advance();
          if (!last_stage) {
            ok = __all_sync(0xffffffffu, bounded_wait(bar_tmem_full + 8 * tm.slot, tm.parity, env, kErrEpilogueWait));
            if (!ok) break;
            tc_fence_after_sync();
            tmem_ld_32x32b_x16_before(t_lane + tm.slot * 2 * kBN, vA, vB[0]);
          }
          if (two) rescale_fragment<DEBUG>(vB, swp + kBN / 4 + 4, sa1, acc + 8, DEBUG && d0 ? d0 + 16 : nullptr);
          if (!last_stage) tmem_wait_ld_after(acc_hi);
          sc.advance();
        }
        if (!ok) break;
        if (p.yref != nullptr) {
          // Eq. 10's objective: || Y_ref - Y_hat ||^2 over the tile, with Y_hat rounded to BF16 exactly as the
          // forward would store it.  FP32 within the thread and the warp, FP64 across warps and tiles.
          float e = 0.0f;
          if (row < p.M) {
            const uint4* yr = reinterpret_cast<const uint4*>(p.yref + static_cast<size_t>(row) * p.N + ch0);
#pragma unroll
            for (int i = 0; i < kEpiCols / 8; ++i) {
              float4 b0 = make_float4(0.f, 0.f, 0.f, 0.f), b1 = b0;
              if (p.bias) {
                b0 = __ldg(reinterpret_cast<const float4*>(p.bias + ch0) + 2 * i);
                b1 = __ldg(reinterpret_cast<const float4*>(p.bias + ch0) + 2 * i + 1);
              }
              const uint4 ref = __ldg(yr + i);
              const float2 a0 = acc[4 * i], a1 = acc[4 * i + 1], a2 = acc[4 * i + 2], a3 = acc[4 * i + 3];
              const float yh[8] = {a0.x + b0.x, a0.y + b0.y, a1.x + b0.z, a1.y + b0.w,
                                   a2.x + b1.x, a2.y + b1.y, a3.x + b1.z, a3.y + b1.w};
              const uint32_t rw[4] = {ref.x, ref.y, ref.z, ref.w};
#pragma unroll
              for (int c = 0; c < 8; ++c) {
                const float y_hat = __bfloat162float(__float2bfloat16_rn(apply_activation(yh[c], p.act)));
                const float y_ref = __uint_as_float((c & 1) ? (rw[c >> 1] & 0xffff0000u) : (rw[c >> 1] << 16));
                const float d = y_ref - y_hat;
                e = fmaf(d, d, e);
              }
            }
          }
#pragma unroll
          for (int o = 16; o > 0; o >>= 1) e += __shfl_xor_sync(0xffffffffu, e, o);
          if (lane == 0) atomicAdd(p.sq_err, static_cast<double>(e));
        } else if (row < p.M) {
          // The thread's channels are contiguous bytes of its output row.
          uint4* yrow = reinterpret_cast<uint4*>(p.Y + static_cast<size_t>(row) * p.N + ch0);
#pragma unroll
          for (int i = 0; i < kEpiCols / 8; ++i) {  // 8 channels per 16-byte store
            float4 b0 = make_float4(0.f, 0.f, 0.f, 0.f), b1 = b0;
            if (p.bias) {
              b0 = __ldg(reinterpret_cast<const float4*>(p.bias + ch0) + 2 * i);
              b1 = __ldg(reinterpret_cast<const float4*>(p.bias + ch0) + 2 * i + 1);
            }
            const float2 a0 = acc[4 * i], a1 = acc[4 * i + 1], a2 = acc[4 * i + 2], a3 = acc[4 * i + 3];
            float y[8] = {a0.x + b0.x, a0.y + b0.y, a1.x + b0.z, a1.y + b0.w, a2.x + b1.x, a2.y + b1.y, a3.x + b1.z, a3.y + b1.w};
            if (p.act != 0) {  // uniform over the grid
#pragma unroll
              for (int c = 0; c < 8; ++c) y[c] = apply_activation(y[c], p.act);
            }
            __nv_bfloat162 o0 = __floats2bfloat162_rn(y[0], y[1]);
            __nv_bfloat162 o1 = __floats2bfloat162_rn(y[2], y[3]);
            __nv_bfloat162 o2 = __floats2bfloat162_rn(y[4], y[5]);
            __nv_bfloat162 o3 = __floats2bfloat162_rn(y[6], y[7]);
            uint4 o;
            o.x = *reinterpret_cast<uint32_t*>(&o0);
            o.y = *reinterpret_cast<uint32_t*>(&o1);
            o.z = *reinterpret_cast<uint32_t*>(&o2);
            o.w = *reinterpret_cast<uint32_t*>(&o3);
            yrow[i] = o;
          }
        }
      }
    }
  }

  // ---------------------------------------------------------------------- common tail
  tc_fence_before_sync();
  __syncthreads();
  if (*s_abort) {
    // Something gave up: give copies that may still be in flight time to land before the CTA's
    // shared memory is released.
    const uint64_t t0 = global_timer_ns();
    while (global_timer_ns() - t0 < 200000ull) __nanosleep(1000);
    __syncthreads();
  }
  if (warp == 2) {
    tc_fence_after_sync();
    tmem_dealloc(tmem_base, 512);
  }
}

}  // namespace w4a4
