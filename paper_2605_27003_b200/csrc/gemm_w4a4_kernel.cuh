// Kernel 2: fused W4A4 GEMM + per-group rescale + low-rank up-projection + bias + BF16 store.
//
//   Eq. 7 / 11    Y[m,n] = sum_g  P_g[m,n] * sx[m,g] * sw[g,n]  +  sum_j T[m,j] L2[j,n]  +  b[n]
//                 P_g[m,n] = sum_{k in group g} q[m,k] qw[k,n]            (exact: integers in FP32)
//
// Code products.  The 4-bit codes go through the tensor core as E4M3 bytes (fp8_codes.cuh): tcgen05.mma
// kind::f8f6f4 runs at the 8-bit rate and leaves every group's partial sums in TMEM as exact integers already in
// FP32 (|P| <= 4096).  The activation codes come straight from kernel 1, the weight codes from
// expand_weight_kernel, which runs right before this kernel and turns the layer's nibble-packed weights (their
// format at rest) into an N x K byte image that stays in L2 for the duration of the GEMM.
//
// Scale products.  The factor S_g = sx[:, g] (x) sw[g, :] is an outer product, i.e. a K = 16 BF16 MMA on operands
// that hold each scale as two BF16 pieces (s = h + m up to 2^-16 relative):
//     token row,   four slots per group:  [h,  h,  m,  m ]
//     channel row, four slots per group:  [w1, w2, w1, w2]      ->  h w1 + h w2 + m w1 + m w2 = sx sw (1 + O(2^-16))
// One 16-byte K chunk of a token row carries the slots of the two groups of a stage; the channel side has one
// chunk per group with zeros in the other group's slots, and every descriptor's second K chunk points at a tile of
// zeros.  The epilogue then needs one fused multiply-add per partial sum, acc += P_g * S_g, on two TMEM fragments
// and reads no scales from shared memory.  Operand tiles of the scale MMA live in global memory as ready-made
// shared-memory images (no-swizzle K-major canonical layout: [8-row group][8 rows][16 bytes]); kernel 1 writes the
// token side next to the FP32 scales, the channel side is built once at pack time.  The low-rank product T L2 goes
// through the same path as one more "group" that opens a tile: its P is the BF16 product [T_hi | T_lo] [L2 | L2]^T,
// its S is the constant 1 (an MMA on a tile of ones), so the epilogue has a single loop.
//
// Persistent, one CTA (640 threads) per SM, 128 x 128 tiles, column tile fastest (the CTAs running at any moment
// share a few row blocks of A and a super-column of B through L2).  TMEM: two slots of 256 columns, one per group in flight:
// columns 0..127 P_g, columns 128..255 S_g.  Warp roles:
//   warp 0      producer: per stage of 128 K-codes (two groups) TMA loads of the A and B code tiles (16 KiB each,
//               128-byte swizzle) and of the two scale-operand images, all onto the stage's mbarrier;
//   warp 1      code-MMA issuer: per group two tcgen05.mma kind::f8f6f4 (K = 32) into the slot's P columns, then a
//               commit onto tmem_full[slot];
//   warp 3      scale-MMA issuer: per group one tcgen05.mma kind::f16 (K = 16) into the slot's S columns and a commit
//               onto the same barrier (it counts two arrivals).  Two issuing threads because the issue of a
//               tcgen05.mma waits for room in the tensor pipe's queue: one thread would put all of that on the
//               hand-over path of every slot;
//   warp 2      TMEM allocation;
//   warps 4-19  epilogue: a thread owns one token row and 32 output channels.  Per group two round trips of two
//               tcgen05.ld.32x32b.x16 (P and S of 16 columns) with the eight packed multiply-adds of the first half
//               in between; the slot goes back to the issuing warps (tmem_empty[slot], 16 arrivals) as soon as the
//               second half is in registers.  Measured alternatives (all four loads in one round trip; the second
//               half's loads issued ahead of the first half's arithmetic; warps of a scheduler skewed against one
//               another) were slower.
// What bounds the kernel is the round trip of a TMEM slot (two slots, so two round trips overlap): epilogue releases it
// -> issuing warps see that -> MMAs run -> commit -> epilogue sees that -> loads.  A lone warp's dependent instructions
// cost 10-15 cycles each and a branch on a fresh mbarrier result ~70, so the hops are written as single instruction
// sequences without branches: wait_issue_* (try_wait, then fence, MMAs and commit predicated on its answer),
// wait_then_ld16 (try_wait, then fence and first TMEM load predicated on its answer), descriptors computed before the wait, and
// predicated instead of branched single-lane instructions (umma_*_if, mbar_arrive_if).  A wait that outlasts the
// try_wait falls back to the bounded wait of pipeline.cuh and the same instructions issued from C++.
// Tile order: column tiles are walked in super-columns (GemmParams::sc_tiles column tiles wide, all row blocks of a
// super-column before the next) sized so that the weight bytes a wave of CTAs touches stay in L2; with the plain
// row-major order the 71 MB weight image of the FFN shapes streamed from DRAM once per 1.4 row blocks.
// Every role loops warp-uniformly (waits are voted, only the TMA / tcgen05 instructions are predicated on one elected
// lane), which keeps ring positions, addresses and descriptors in uniform registers.  All waits are bounded
// (pipeline.cuh).  Finally + bias -> optional GELU -> BF16, or the squared error against a reference (clip search).
#pragma once

#include <cuda_bf16.h>
#include <stdint.h>

#include "pipeline.cuh"
#include "ptx.cuh"

namespace w4a4 {

constexpr int kGemmStages = 5;
constexpr int kTmemSlots = 2;       // TMEM slots of 2 x kBN columns: one per group in flight
constexpr uint32_t kOpATile = kBM * kBK;              // 16 KiB: 128 token rows x 128 codes
constexpr uint32_t kOpBTile = kBN * kBK;              // 16 KiB: 128 weight rows x 128 codes
constexpr uint32_t kSopATile = kBM * 16;              // 2 KiB: 128 token rows x one 16-byte chunk (two groups)
constexpr uint32_t kSopBTile = 2 * kBN * 16;          // 4 KiB: per group 128 channel rows x one 16-byte chunk
constexpr uint32_t kStageBytes = kOpATile + kOpBTile + kSopATile + kSopBTile;   // 38 KiB
constexpr uint32_t kLrStageBytes = kOpATile + kOpBTile;   // a low-rank stage: T tile and L2 rows
constexpr uint32_t kConstTile = 2048;                 // tiles of zeros and of ones: 128 rows x 16 bytes
constexpr uint32_t kGemmNumBarriers = 2 * kGemmStages + 2 * kTmemSlots;
constexpr uint32_t kGemmSmemBytes = 1024 + kGemmStages * kStageBytes + 2 * kConstTile + kGemmNumBarriers * 8 + 16;
static_assert(kGemmSmemBytes <= 232448, "shared memory budget of one CTA");
static_assert(kStageBytes % 1024 == 0, "operand tiles must stay 1024-byte aligned");

// Register budgets: the launch bound fixes 96 registers per thread for all 20 warps (five per scheduler: one control
// warp and four epilogue warps).  Moving registers from the control warps to the epilogue with setmaxnreg was
// measured and does not pay: at 104 the time is the same, at 112 the compiler's freer scheduling of the TMEM loads
// against the multiply-adds made the kernel 7 % slower.

// Wait for a TMEM slot and issue its MMAs in one branch-free instruction sequence: one try_wait (it blocks in hardware
// for a while before it gives up), then the fence, the MMAs and the commit predicated on its answer.  A branch on the
// fresh answer would hold the warp ~70 cycles; a second try_wait predicated on the first one's failure costs its
// latency even when it is skipped (both measured slower).  Returns 0 if the barrier did not complete (the caller then
// takes the bounded wait and issues from C++).
__device__ __forceinline__ uint32_t wait_issue_f8x2(uint32_t go, uint32_t bar, uint32_t parity, uint32_t d_tmem, uint64_t a0, uint64_t b0,
                                                    uint64_t a1, uint64_t b1, uint32_t idesc, uint32_t full_bar) {
  uint32_t done;
  asm volatile(
      "{\n"
      ".reg .pred p, q, pq;\n"
      "setp.ne.b32 q, %6, 0;\n"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
      "and.pred pq, p, q;\n"
      "@p tcgen05.fence::after_thread_sync;\n"
      "@pq tcgen05.mma.cta_group::1.kind::f8f6f4 [%3], %4, %5, %7, 0;\n"
      "@pq tcgen05.mma.cta_group::1.kind::f8f6f4 [%3], %8, %9, %7, 1;\n"
      "@pq tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%10];\n"
      "selp.u32 %0, 1, 0, p;\n"
      "}\n"
      : "=r"(done)
      : "r"(bar), "r"(parity), "r"(d_tmem), "l"(a0), "l"(b0), "r"(go), "r"(idesc), "l"(a1), "l"(b1), "r"(full_bar)
      : "memory");
  return done;
}
__device__ __forceinline__ uint32_t wait_issue_f16(uint32_t go, uint32_t bar, uint32_t parity, uint32_t d_tmem, uint64_t a0, uint64_t b0,
                                                   uint32_t idesc, uint32_t full_bar) {
  uint32_t done;
  asm volatile(
      "{\n"
      ".reg .pred p, q, pq;\n"
      "setp.ne.b32 q, %6, 0;\n"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
      "and.pred pq, p, q;\n"
      "@p tcgen05.fence::after_thread_sync;\n"
      "@pq tcgen05.mma.cta_group::1.kind::f16 [%3], %4, %5, %7, 0;\n"
      "@pq tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%8];\n"
      "selp.u32 %0, 1, 0, p;\n"
      "}\n"
      : "=r"(done)
      : "r"(bar), "r"(parity), "r"(d_tmem), "l"(a0), "l"(b0), "r"(go), "r"(idesc), "r"(full_bar)
      : "memory");
  return done;
}

// Wait for a full TMEM slot and start its first load in one branch-free instruction sequence.  Returns 0 if the barrier
// did not complete within the try_wait (nothing was loaded then).
__device__ __forceinline__ uint32_t wait_then_ld16(uint32_t bar, uint32_t parity, uint32_t taddr, uint32_t (&v)[16]) {
  uint32_t done;
  asm volatile(
      "{\n"
      ".reg .pred p;\n"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%17], %18;\n"
      "@p tcgen05.fence::after_thread_sync;\n"
      "@p tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%19];\n"
      "selp.u32 %16, 1, 0, p;\n"
      "}\n"
      : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]),
        "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]), "=r"(done)
      : "r"(bar), "r"(parity), "r"(taddr)
      : "memory");
  return done;
}

// Tile raster: column tiles are walked in super-columns of `sc` tiles (all row blocks of one super-column before the
// next), so that the weight bytes a wave of CTAs touches stay in L2.  sc == tiles_n: plain row-major order.
__device__ __forceinline__ void tile_coords(int tile, int tiles_m, int tiles_n, int sc, int& tm, int& tn) {
  const int per_sc = tiles_m * sc;
  const int full = tiles_n / sc;
  int s_idx = tile / per_sc, rem = tile - s_idx * per_sc, width = sc;
  if (s_idx >= full) {
    s_idx = full;
    rem = tile - full * per_sc;
    width = tiles_n - full * sc;
  }
  tm = rem / width;
  tn = s_idx * sc + (rem - tm * width);
}

// Ties a fragment to the tcgen05.wait::ld in front of it: the registers count as written there, so nothing that
// reads them can be scheduled above the wait (an asm statement takes at most 30 operands, hence one statement per
// fragment; volatile statements keep their order).
__device__ __forceinline__ void tie_fragment(uint32_t (&a)[16]) {
  asm volatile(""
               : "+r"(a[0]), "+r"(a[1]), "+r"(a[2]), "+r"(a[3]), "+r"(a[4]), "+r"(a[5]), "+r"(a[6]), "+r"(a[7]), "+r"(a[8]),
                 "+r"(a[9]), "+r"(a[10]), "+r"(a[11]), "+r"(a[12]), "+r"(a[13]), "+r"(a[14]), "+r"(a[15])
               :
               : "memory");
}

// acc[j] += P * S for the fragment's eight column pairs.
template <bool DEBUG>
__device__ __forceinline__ void fma_fragment(const uint32_t (&pv)[16], const uint32_t (&sv)[16], float2* acc, int32_t* dbg_row) {
#pragma unroll
  for (int j = 0; j < 8; ++j) {
    const float2 p2 = make_float2(__uint_as_float(pv[2 * j]), __uint_as_float(pv[2 * j + 1]));
    const float2 s2 = make_float2(__uint_as_float(sv[2 * j]), __uint_as_float(sv[2 * j + 1]));
    acc[j] = __ffma2_rn(p2, s2, acc[j]);
    if (DEBUG) {
      if (dbg_row != nullptr) {
        dbg_row[2 * j] = static_cast<int32_t>(p2.x);
        dbg_row[2 * j + 1] = static_cast<int32_t>(p2.y);
      }
    }
  }
}

// One scale as two BF16 pieces: s = h + m up to 2^-16 relative.
__device__ __forceinline__ uint32_t scale_pieces(float s) {
  const __nv_bfloat16 h = __float2bfloat16_rn(s);
  const __nv_bfloat16 m = __float2bfloat16_rn(s - __bfloat162float(h));
  return static_cast<uint32_t>(__bfloat16_as_ushort(h)) | (static_cast<uint32_t>(__bfloat16_as_ushort(m)) << 16);
}

// Weight-side scale operands of one expert (run once per layer): wscale [G, N] FP32 -> per (128 channels, stage) one
// 4 KiB image [group of the stage][8-row group][8 rows][16 bytes]; the chunk of group parity v holds
// [w1, w2, w1, w2] in slots 4 v .. 4 v + 3 and zeros in the other group's slots.  `out` is zero-filled beforehand.
__global__ void sop_weight_kernel(const float* __restrict__ wscale, uint4* __restrict__ out, int G, int N) {
  const size_t i = static_cast<size_t>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (i >= static_cast<size_t>(G) * N) return;
  const int g = static_cast<int>(i / N), n = static_cast<int>(i % N);
  const uint32_t w = scale_pieces(wscale[i]);
  const int stages = (G + 1) >> 1;
  const size_t image = static_cast<size_t>(n >> 7) * stages + (g >> 1);
  out[image * 256 + (g & 1) * 128 + ((n & 127) >> 3) * 8 + (n & 7)] = (g & 1) ? make_uint4(0u, 0u, w, w) : make_uint4(w, w, 0u, 0u);
}

template <bool DEBUG>
__global__ void __launch_bounds__(kGemmThreads, 1)
gemm_w4a4_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                 const __grid_constant__ CUtensorMap tmT, const __grid_constant__ CUtensorMap tmL2,
                 const __grid_constant__ CUtensorMap tmSopA, const __grid_constant__ CUtensorMap tmSopB, const GemmParams p) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* smem = smem_raw + (smem_base - smem_u32(smem_raw));
  // Constant tiles, above every operand tile so that the descriptors' chunk distances are positive.
  const uint32_t ones_base = smem_base + kGemmStages * kStageBytes;   // rows [1, 0, 0, 0, 0, 0, 0, 0]: S = 1 for the low-rank entry
  const uint32_t zero_base = ones_base + kConstTile;                  // second K chunk of every scale MMA
  const uint32_t bar_base = zero_base + kConstTile;
  const uint32_t bar_op_full = bar_base;
  const uint32_t bar_op_empty = bar_op_full + 8 * kGemmStages;
  const uint32_t bar_tmem_full = bar_op_empty + 8 * kGemmStages;
  const uint32_t bar_tmem_empty = bar_tmem_full + 8 * kTmemSlots;
  const uint32_t misc_off = (bar_tmem_empty + 8 * kTmemSlots) - smem_base;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + misc_off);
  volatile int* s_abort = reinterpret_cast<volatile int*>(smem + misc_off + 4);

  const int warp = __shfl_sync(0xffffffffu, static_cast<int>(threadIdx.x >> 5), 0), lane = threadIdx.x & 31;  // provably warp-uniform
  const int G = p.K >> 6;
  const int n_int_stages = (G + 1) >> 1;
  const int n_lr_stages = p.r > 0 ? (2 * p.r + 63) / 64 : 0;
  const int num_tiles = p.tiles_m * p.tiles_n;
  const int sc_tiles = p.sc_tiles;
  const WaitEnv env{p.err, s_abort, p.wait_limit_ns};

  if (threadIdx.x == 0) {
    *s_abort = (*reinterpret_cast<volatile int*>(p.err) != 0) ? 1 : 0;
    for (int i = 0; i < kGemmStages; ++i) {
      mbar_init(bar_op_full + 8 * i, 1);
      mbar_init(bar_op_empty + 8 * i, 2);    // the code-MMA warp and the scale-MMA warp
    }
    for (int i = 0; i < kTmemSlots; ++i) {
      mbar_init(bar_tmem_full + 8 * i, 2);   // the code-MMA warp and the scale-MMA warp
      mbar_init(bar_tmem_empty + 8 * i, kEpiWarps);
    }
    mbar_fence_init();
    fence_proxy_async_smem();
    tma_prefetch_desc(&tmA);
    tma_prefetch_desc(&tmB);
    tma_prefetch_desc(&tmSopA);
    tma_prefetch_desc(&tmSopB);
    if (p.r > 0) {
      tma_prefetch_desc(&tmT);
      tma_prefetch_desc(&tmL2);
    }
  }
  for (uint32_t i = threadIdx.x; i < 2 * kConstTile / 16; i += blockDim.x)
    reinterpret_cast<uint4*>(smem + (ones_base - smem_base))[i] = i < kConstTile / 16 ? make_uint4(0x3F80u, 0u, 0u, 0u) : make_uint4(0u, 0u, 0u, 0u);
  fence_proxy_async_smem();   // the tensor core reads these tiles through the async proxy
  if (warp == 2) {
    tmem_alloc(smem_u32(tmem_slot), 512);
    tmem_relinquish();
    tc_fence_before_sync();
  }
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = __shfl_sync(0xffffffffu, *tmem_slot, 0);
  const bool live = __all_sync(0xffffffffu, *s_abort == 0);

  // Shared-memory stage: A codes | B codes | token scale operand (two groups) | channel scale operand (two groups).
  // Per tile the issuing warps and the epilogue walk the same list of TMEM slot uses: [the low-rank entry, if r > 0]
  // followed by one entry per group.
  if (warp < kEpiWarp0) {
    if (live && warp == 0) {
      // ------------------------------------------------------------------ TMA producer (all lanes loop, one issues)
      const bool issuer = elect_one_lane();
      Ring<kGemmStages> op;
      bool ok = true;
      int stage_no = 0;
      for (int tile = blockIdx.x; ok && tile < num_tiles; tile += gridDim.x) {
        int tm, tn;
        tile_coords(tile, p.tiles_m, p.tiles_n, sc_tiles, tm, tn);
        const int m0 = tm * kBM, n0 = tn * kBN;
        for (int st = 0; st < n_lr_stages + n_int_stages; ++st) {
          ok = __all_sync(0xffffffffu, bounded_wait<64>(bar_op_empty + 8 * op.slot, op.parity ^ 1u, env, kErrProducerWait));
          if (!ok) break;
          if (DEBUG) {
            // Test hook: one stage is never loaded, so its consumers' waits run into their limit and every role of
            // the CTA leaves through the common tail (error word, drain, TMEM release).
            if (stage_no++ == p.dbg_stall_stage) {
              op.advance();
              continue;
            }
          }
          const uint32_t full = bar_op_full + 8 * op.slot;
          const uint32_t dst = smem_base + op.slot * kStageBytes;
          if (st < n_lr_stages) {
            if (issuer) {
              mbar_arrive_expect_tx(full, kLrStageBytes);
              tma_load_2d(dst, &tmT, full, st * 64, m0);
              tma_load_2d(dst + kOpATile, &tmL2, full, st * 64, n0);
            }
          } else if (issuer) {
            const int ks = st - n_lr_stages;
            const uint32_t sop = dst + kOpATile + kOpBTile;
            mbar_arrive_expect_tx(full, kStageBytes);
            tma_load_2d(dst, &tmA, full, ks * kBK, m0);
            tma_load_2d(dst + kOpATile, &tmB, full, ks * kBK, n0);
            // scale operand images as rows of 32-bit words, 256 words (1 KiB) per box
            tma_load_2d(sop, &tmSopA, full, ks * 512, tm);
            tma_load_2d(sop + 1024, &tmSopA, full, ks * 512 + 256, tm);
#pragma unroll
            for (int c = 0; c < 4; ++c) tma_load_2d(sop + kSopATile + 1024 * c, &tmSopB, full, ks * 1024 + 256 * c, tn);
          }
          op.advance();
        }
      }
    } else if (live && warp == 1) {
      // ------------------------------------------------------------------ code-MMA issuer (all lanes loop, one issues)
      constexpr uint32_t idesc_f8 = umma_idesc(1, 0, kBM, kBN);
      constexpr uint32_t idesc_bf16 = umma_idesc(1, 1, kBM, kBN);
      const bool issuer = elect_one_lane();
      const uint32_t go = issuer ? 1u : 0u;
      const int issue_lane = __ffs(__ballot_sync(0xffffffffu, issuer)) - 1;   // the decision below is the issuing lane's
      Ring<kGemmStages> op;
      Ring<kTmemSlots> tm;
      bool ok = true;
      for (int tile = blockIdx.x; ok && tile < num_tiles; tile += gridDim.x) {
        if (n_lr_stages > 0) {
          ok = __all_sync(0xffffffffu, bounded_wait<0, 1>(bar_tmem_empty + 8 * tm.slot, tm.parity ^ 1u, env, kErrMmaWait));
          if (ok) tc_fence_after_sync();
          const uint32_t d = tmem_base + tm.slot * 2 * kBN;
          const uint32_t full_bar = bar_tmem_full + 8 * tm.slot;
          tm.advance();
          for (int l = 0; ok && l < n_lr_stages; ++l) {
            ok = __all_sync(0xffffffffu, bounded_wait<0, 1>(bar_op_full + 8 * op.slot, op.parity, env, kErrMmaWait));
            if (!ok) break;
            const uint32_t a = smem_base + op.slot * kStageBytes, b = a + kOpATile;
            if (issuer) {
#pragma unroll
              for (int kk = 0; kk < 4; ++kk)
                umma_f16(d, umma_desc_k_sw128(a, 32 * kk), umma_desc_k_sw128(b, 32 * kk), idesc_bf16, (l > 0 || kk > 0) ? 1u : 0u);
              umma_commit(bar_op_empty + 8 * op.slot);
            }
            op.advance();
          }
          if (!ok) break;
          if (issuer) umma_commit(full_bar);
        }
        for (int st = 0; ok && st < n_int_stages; ++st) {
          ok = __all_sync(0xffffffffu, bounded_wait<0, 1>(bar_op_full + 8 * op.slot, op.parity, env, kErrMmaWait));
          if (!ok) break;
          const uint32_t a = smem_base + op.slot * kStageBytes, b = a + kOpATile;
          const int groups = (2 * st + 1 < G) ? 2 : 1;
          for (int v = 0; v < groups; ++v) {
            // everything the issue needs is ready before the wait that sits on the slot's round trip
            const uint32_t d = tmem_base + tm.slot * 2 * kBN;
            const uint32_t full_bar = bar_tmem_full + 8 * tm.slot;
            const uint64_t da0 = umma_desc_k_sw128(a, 64 * v), db0 = umma_desc_k_sw128(b, 64 * v);
            const uint64_t da1 = umma_desc_k_sw128(a, 64 * v + 32), db1 = umma_desc_k_sw128(b, 64 * v + 32);
            if (__shfl_sync(0xffffffffu, wait_issue_f8x2(go, bar_tmem_empty + 8 * tm.slot, tm.parity ^ 1u, d, da0, db0, da1, db1, idesc_f8, full_bar), issue_lane) == 0) {
              ok = __all_sync(0xffffffffu, bounded_wait<0, 1>(bar_tmem_empty + 8 * tm.slot, tm.parity ^ 1u, env, kErrMmaWait));
              if (!ok) break;
              tc_fence_after_sync();
              umma_f8_if(go, d, da0, db0, idesc_f8, 0u);
              umma_f8_if(go, d, da1, db1, idesc_f8, 1u);
              umma_commit_if(go, full_bar);
            }
            tm.advance();
          }
          if (!ok) break;
          umma_commit_if(go, bar_op_empty + 8 * op.slot);
          op.advance();
        }
      }
    } else if (live && warp == 3) {
      // ------------------------------------------------------------------ scale-MMA issuer
      // Walks the same slot uses as the code-MMA warp: S = 1 for the low-rank entry, S_g for the groups.
      constexpr uint32_t idesc_bf16 = umma_idesc(1, 1, kBM, kBN);
      const bool issuer = elect_one_lane();
      const uint32_t go = issuer ? 1u : 0u;
      const int issue_lane = __ffs(__ballot_sync(0xffffffffu, issuer)) - 1;   // the decision below is the issuing lane's
      Ring<kGemmStages> op;
      Ring<kTmemSlots> tm;
      bool ok = true;
      for (int tile = blockIdx.x; ok && tile < num_tiles; tile += gridDim.x) {
        if (n_lr_stages > 0) {
          ok = __all_sync(0xffffffffu, bounded_wait<0, 1>(bar_tmem_empty + 8 * tm.slot, tm.parity ^ 1u, env, kErrMmaWait));
          if (!ok) break;
          tc_fence_after_sync();
          if (issuer) {
            const uint64_t ones = umma_desc_k_plain(ones_base, zero_base - ones_base, 128);
            umma_f16(tmem_base + tm.slot * 2 * kBN + kBN, ones, ones, idesc_bf16, 0u);
            umma_commit(bar_tmem_full + 8 * tm.slot);
          }
          tm.advance();
          for (int l = 0; ok && l < n_lr_stages; ++l) {   // the low-rank stages hold nothing for this warp: sign off
            ok = __all_sync(0xffffffffu, bounded_wait<0, 1>(bar_op_full + 8 * op.slot, op.parity, env, kErrMmaWait));
            if (!ok) break;
            if (issuer) mbar_arrive(bar_op_empty + 8 * op.slot);
            op.advance();
          }
          if (!ok) break;
        }
        for (int st = 0; ok && st < n_int_stages; ++st) {
          ok = __all_sync(0xffffffffu, bounded_wait<0, 1>(bar_op_full + 8 * op.slot, op.parity, env, kErrMmaWait));
          if (!ok) break;
          const uint32_t sa = smem_base + op.slot * kStageBytes + kOpATile + kOpBTile, sb = sa + kSopATile;
          const int groups = (2 * st + 1 < G) ? 2 : 1;
          for (int v = 0; v < groups; ++v) {
            const uint32_t d = tmem_base + tm.slot * 2 * kBN + kBN;
            const uint32_t full_bar = bar_tmem_full + 8 * tm.slot;
            const uint32_t cb = sb + (kSopBTile / 2) * v;   // the channel side's chunk of this group
            const uint64_t dsa = umma_desc_k_plain(sa, zero_base - sa, 128), dsb = umma_desc_k_plain(cb, zero_base - cb, 128);
            if (__shfl_sync(0xffffffffu, wait_issue_f16(go, bar_tmem_empty + 8 * tm.slot, tm.parity ^ 1u, d, dsa, dsb, idesc_bf16, full_bar), issue_lane) == 0) {
              ok = __all_sync(0xffffffffu, bounded_wait<0, 1>(bar_tmem_empty + 8 * tm.slot, tm.parity ^ 1u, env, kErrMmaWait));
              if (!ok) break;
              tc_fence_after_sync();
              umma_f16_if(go, d, dsa, dsb, idesc_bf16, 0u);
              umma_commit_if(go, full_bar);
            }
            tm.advance();
          }
          if (!ok) break;
          umma_commit_if(go, bar_op_empty + 8 * op.slot);
          op.advance();
        }
      }
    }
  } else {
    if (live) {
      // ------------------------------------------------------------------ epilogue warps
      // Warp ew owns TMEM lanes 32 * (ew % 4) .. +31 (token rows) and the 32-column block ew / 4; a thread owns one
      // row and the block's 32 output channels.
      const int ew = warp - kEpiWarp0;
      const int quarter = ew & 3, colblk = ew >> 2;
      const uint32_t t_lane = tmem_base + (static_cast<uint32_t>(32 * quarter) << 16) + kEpiCols * colblk;
      const int entries = G + (n_lr_stages > 0 ? 1 : 0);
      Ring<kTmemSlots> tm;
      bool ok = true;
      for (int tile = blockIdx.x; ok && tile < num_tiles; tile += gridDim.x) {
        int tm_e, tn_e;
        tile_coords(tile, p.tiles_m, p.tiles_n, sc_tiles, tm_e, tn_e);
        const int m0 = tm_e * kBM, n0 = tn_e * kBN;
        const bool dbg_tile = DEBUG && p.dbg_P != nullptr && m0 == p.dbg_m0 && n0 == p.dbg_n0;
        float2 acc[16];  // pair k: channels ch0 + 2 k, ch0 + 2 k + 1
#pragma unroll
        for (int j = 0; j < 16; ++j) acc[j] = make_float2(0.0f, 0.0f);
        for (int e = 0; e < entries; ++e) {
          const uint32_t t = t_lane + tm.slot * 2 * kBN;
          uint32_t pv[16], sv[16];
          if (!__all_sync(0xffffffffu, wait_then_ld16(bar_tmem_full + 8 * tm.slot, tm.parity, t, pv) != 0)) {
            ok = __all_sync(0xffffffffu, bounded_wait(bar_tmem_full + 8 * tm.slot, tm.parity, env, kErrEpilogueWait));
            if (!ok) break;
            tc_fence_after_sync();
            tmem_ld_32x32b_x16(t, pv);
          }
          int32_t* d0 = nullptr;
          if (DEBUG) {
            const int g = e - (n_lr_stages > 0 ? 1 : 0);
            if (dbg_tile && g >= 0) d0 = p.dbg_P + (static_cast<size_t>(32 * quarter + lane) * G + g) * kBN + kEpiCols * colblk;
          }
          tmem_ld_32x32b_x16(t + kBN, sv);
          tmem_wait_ld();
          tie_fragment(pv);
          tie_fragment(sv);
          fma_fragment<DEBUG>(pv, sv, acc, d0);
          tmem_ld_32x32b_x16(t + 16, pv);
          tmem_ld_32x32b_x16(t + kBN + 16, sv);
          tmem_wait_ld();
          tie_fragment(pv);
          tie_fragment(sv);
          // The whole slot is in registers: hand it back to the MMA warps.
          tc_fence_before_sync();
          __syncwarp();
          mbar_arrive_if(lane == 0 ? 1u : 0u, bar_tmem_empty + 8 * tm.slot);
          tm.advance();
          fma_fragment<DEBUG>(pv, sv, acc + 8, DEBUG && d0 ? d0 + 16 : nullptr);
        }
        if (!ok) break;
        const int row = m0 + 32 * quarter + lane;
        const int ch0 = n0 + kEpiCols * colblk;
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
      tmem_wait_ld();   // a role that gave up may still have loads in flight
    }
  }

  // ---------------------------------------------------------------------- common tail
  tc_fence_before_sync();
  __syncthreads();
  drain_after_abort(s_abort);
  if (warp == 2) {
    tc_fence_after_sync();
    tmem_dealloc(tmem_base, 512);
  }
}

}  // namespace w4a4
