// Kernel 2, second form: the INT4-exact GEMM whose per-group rescale factors come out of the tensor core too.
//
// Eq. 7's main term is  sum_g  sx[m, g] * sw[g, n] * P_g[m, n]  with P_g the exact integer partial sum of group g.
// gemm_kernel (gemm_kernel.cuh) multiplies P_g by both scales on the CUDA cores: two FP32 instructions per partial
// sum plus broadcast loads of the weight scales, which is what bounds it.  Here the factor S_g = sx[:, g] (x) sw[g, :]
// is an outer product, i.e. a K = 16 BF16 MMA on operands that hold the two scales split into BF16 pieces:
//     A row (token m, one 8-slot chunk per group):    [h, h, h, m, m, m, l, l]     sx = h + m + l  (BF16 each)
//     B row (channel n, one 8-slot chunk per group):  [w1, w2, w3, w1, w2, w3, w1, w2]   sw = w1 + w2 + w3
// so that the MMA's FP32 sum is  h w1 + h w2 + h w3 + m w1 + m w2 + m w3 + l w1 + l w2 = sx * sw  up to the
// dropped term l w3 (below 2^-24 of the product) and the FP32 summation.  A K = 16 operand row carries the chunks of the
// two groups of a stage; the MMA of one group starts both descriptors at that group's chunk and points their second
// K chunk at a tile of zeros.  The epilogue then does one fused multiply-add per partial sum, acc += P_g * S_g, on two
// TMEM fragments, and reads no scales from shared memory at all.
//
// Operand tiles of the scale MMA are stored in global memory as ready-made 4 KiB shared-memory images (no-swizzle
// K-major canonical layout: [8-row group][K chunk][8 rows][16 bytes]) and fetched with plain bulk copies.
//
// TMEM: two slots of 256 columns, one per group in flight: columns 0..127 P_g (or T L2 for the low-rank slot),
// columns 128..255 S_g.  With a group per slot the MMA side's issue time sits on the hand-over path (a thread needs
// some 40 cycles per tcgen05 instruction), so two warps issue: warp 1 the code MMAs, warp 3 the scale MMAs; both wait
// for the same barriers and both commit (op_empty and tmem_full count two arrivals).  Other roles, barriers and
// bounded waits as in gemm_kernel.cuh.
#pragma once

#include <cuda_bf16.h>
#include <stdint.h>

#include "gemm_kernel.cuh"
#include "ptx.cuh"

namespace w4a4 {

constexpr int kOsStages = 5;
constexpr uint32_t kOsSopTile = kBM * 32;   // 4 KiB: 128 rows x 16 BF16 slots
constexpr uint32_t kOsStageBytes = kOpATile + kOpBTile + 2 * kOsSopTile;   // A, B, scale operands of the tokens and of the channels
constexpr uint32_t kOsNumBarriers = 2 * kOsStages + 2 * kTmemSlots;
constexpr uint32_t kOsSmemBytes = 1024 + kOsStages * kOsStageBytes + kOsSopTile /* zeros */ + kOsNumBarriers * 8 + 16;
static_assert(kOsSmemBytes <= 232448, "shared memory budget of one CTA");
static_assert(kOsStageBytes % 1024 == 0, "operand tiles must stay 1024-byte aligned");

// Shared-memory descriptor of a scale-operand tile: K-major, no swizzle, the two 16-byte K chunks of a row group
// 128 bytes apart (leading byte offset), 8-row groups 256 bytes apart (stride byte offset).
// `second_chunk` is the byte distance from the first K chunk (8 slots) of a row group to the second one.  A scale
// operand row carries the chunks of the two groups of a stage next to each other; the MMA of one group starts its
// descriptor at that group's chunk and points the second chunk at a tile of zeros, so that only that group's eight
// products are summed.
__device__ __forceinline__ uint64_t sop_desc(uint32_t smem_addr, uint32_t second_chunk) {
  uint64_t d = 0;
  d |= static_cast<uint64_t>((smem_addr >> 4) & 0x3FFFu);
  d |= static_cast<uint64_t>((second_chunk >> 4) & 0x3FFFu) << 16;
  d |= static_cast<uint64_t>(256u >> 4) << 32;
  d |= static_cast<uint64_t>(1u) << 46;
  return d;
}

__device__ __forceinline__ void bulk_load_g2s(uint32_t dst_smem, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst_smem),
               "l"(src), "r"(bytes), "r"(bar)
               : "memory");
}

// tcgen05.wait::ld for two 16-register fragments (an asm statement takes at most 30 operands: the second fragment is
// tied by an empty statement right behind the wait).
__device__ __forceinline__ void tmem_wait_ld_into(uint32_t (&a)[16], uint32_t (&b)[16]) {
  asm volatile("tcgen05.wait::ld.sync.aligned;"
               : "+r"(a[0]), "+r"(a[1]), "+r"(a[2]), "+r"(a[3]), "+r"(a[4]), "+r"(a[5]), "+r"(a[6]), "+r"(a[7]), "+r"(a[8]),
                 "+r"(a[9]), "+r"(a[10]), "+r"(a[11]), "+r"(a[12]), "+r"(a[13]), "+r"(a[14]), "+r"(a[15])
               :
               : "memory");
  asm volatile(""
               : "+r"(b[0]), "+r"(b[1]), "+r"(b[2]), "+r"(b[3]), "+r"(b[4]), "+r"(b[5]), "+r"(b[6]), "+r"(b[7]), "+r"(b[8]),
                 "+r"(b[9]), "+r"(b[10]), "+r"(b[11]), "+r"(b[12]), "+r"(b[13]), "+r"(b[14]), "+r"(b[15])
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

// Weight-side scale operands of one expert (run once per layer): wscale [G, N] FP32 -> for every (column tile,
// stage) two 4 KiB images; image v holds the chunks of group 2 stage + v and zeros in the other group's slots.
// `out` is zero-filled beforehand.  Chunk: s = w1 + w2 + w3 -> [w1, w2, w3, w1, w2, w3, w1, w2].
__global__ void sop_weight_kernel(const float* __restrict__ wscale, uint4* __restrict__ out, int G, int N) {
  const size_t i = static_cast<size_t>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (i >= static_cast<size_t>(G) * N) return;
  const int g = static_cast<int>(i / N), n = static_cast<int>(i % N);
  const float s = wscale[i];
  const __nv_bfloat16 w1 = __float2bfloat16_rn(s);
  const float r1 = s - __bfloat162float(w1);
  const __nv_bfloat16 w2 = __float2bfloat16_rn(r1);
  const __nv_bfloat16 w3 = __float2bfloat16_rn(r1 - __bfloat162float(w2));
  const uint32_t a = __bfloat16_as_ushort(w1), b = __bfloat16_as_ushort(w2), c = __bfloat16_as_ushort(w3);
  const int stages = (G + 1) >> 1;
  const size_t image = static_cast<size_t>(n >> 7) * stages + (g >> 1);
  out[image * 256 + ((n & 127) >> 3) * 16 + (g & 1) * 8 + (n & 7)] = make_uint4(a | (b << 16), c | (a << 16), b | (c << 16), a | (b << 16));
}

struct OsParams {
  const uint8_t* a_sop;   // activation scale operands: [ceil(M/128)][stages][4096]
  const uint8_t* b_sop;   // weight scale operands:     [N/128][stages][4096]
};

template <bool DEBUG>
__global__ void __launch_bounds__(kGemmThreads, 1)
gemm_os_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
               const __grid_constant__ CUtensorMap tmT, const __grid_constant__ CUtensorMap tmL2, const GemmParams p,
               const OsParams q) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* smem = smem_raw + (smem_base - smem_u32(smem_raw));
  const uint32_t zero_base = smem_base + kOsStages * kOsStageBytes;   // 4 KiB of zeros: the "other group" of a scale MMA
  const uint32_t bar_base = zero_base + kOsSopTile;
  const uint32_t bar_op_full = bar_base;
  const uint32_t bar_op_empty = bar_op_full + 8 * kOsStages;
  const uint32_t bar_tmem_full = bar_op_empty + 8 * kOsStages;
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
    for (int i = 0; i < kOsStages; ++i) {
      mbar_init(bar_op_full + 8 * i, 1);
      mbar_init(bar_op_empty + 8 * i, 2);    // the code-MMA warp and the scale-MMA warp
    }
    for (int i = 0; i < kTmemSlots; ++i) {
      mbar_init(bar_tmem_full + 8 * i, 2);
      mbar_init(bar_tmem_empty + 8 * i, kEpiWarps);
    }
    mbar_fence_init();
    fence_proxy_async_smem();
    tma_prefetch_desc(&tmA);
    tma_prefetch_desc(&tmB);
    if (p.r > 0) {
      tma_prefetch_desc(&tmT);
      tma_prefetch_desc(&tmL2);
    }
  }
  for (uint32_t i = threadIdx.x; i < kOsSopTile / 16; i += blockDim.x)
    reinterpret_cast<uint4*>(smem + (zero_base - smem_base))[i] = make_uint4(0u, 0u, 0u, 0u);
  fence_proxy_async_smem();   // the tensor core reads these zeros through the async proxy
  if (warp == 2) {
    tmem_alloc(smem_u32(tmem_slot), 512);
    tmem_relinquish();
    tc_fence_before_sync();
  }
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = __shfl_sync(0xffffffffu, *tmem_slot, 0);
  const bool live = __all_sync(0xffffffffu, *s_abort == 0);

  if (warp < kEpiWarp0) {
    set_max_regs_dec<kRegsControl>();
    if (live && warp == 0) {
      // ------------------------------------------------------------------ TMA producer (all lanes loop, one issues)
      // Stage: A codes | B codes | scale operand of the 128 tokens | scale operand of the 128 channels.
      const bool issuer = elect_one_lane();
      Ring<kOsStages> op;
      bool ok = true;
      for (int tile = blockIdx.x; ok && tile < num_tiles; tile += gridDim.x) {
        const int tm = tile / p.tiles_n, tn = tile % p.tiles_n;
        const int m0 = tm * kBM, n0 = tn * kBN;
        for (int st = 0; st < n_lr_stages + n_int_stages; ++st) {
          ok = __all_sync(0xffffffffu, bounded_wait<128>(bar_op_empty + 8 * op.slot, op.parity ^ 1u, env, kErrProducerWait));
          if (!ok) break;
          const uint32_t full = bar_op_full + 8 * op.slot;
          const uint32_t dst = smem_base + op.slot * kOsStageBytes;
          if (st < n_lr_stages) {
            if (issuer) {
              mbar_arrive_expect_tx(full, kOpATile + kOpBTile);
              tma_load_2d(dst, &tmT, full, st * 64, m0);
              tma_load_2d(dst + kOpATile, &tmL2, full, st * 64, n0);
            }
          } else if (issuer) {
            const int ks = st - n_lr_stages;
            mbar_arrive_expect_tx(full, kOsStageBytes);
            tma_load_2d(dst, &tmA, full, ks * kBK, m0);
            tma_load_2d(dst + kOpATile, &tmB, full, ks * kBK, n0);
            bulk_load_g2s(dst + kOpATile + kOpBTile, q.a_sop + (static_cast<size_t>(tm) * n_int_stages + ks) * kOsSopTile, kOsSopTile, full);
            bulk_load_g2s(dst + kOpATile + kOpBTile + kOsSopTile, q.b_sop + (static_cast<size_t>(tn) * n_int_stages + ks) * kOsSopTile,
                          kOsSopTile, full);
          }
          op.advance();
        }
      }
    } else if (live && warp == 1) {
      // ------------------------------------------------------------------ MMA issuer (all lanes loop, one issues)
      constexpr uint32_t idesc_f8 = umma_idesc(1, 0, kBM, kBN);
      constexpr uint32_t idesc_bf16 = umma_idesc(1, 1, kBM, kBN);
      const bool issuer = elect_one_lane();
      Ring<kOsStages> op;
      Ring<kTmemSlots> tm;
      bool ok = true;
      for (int tile = blockIdx.x; ok && tile < num_tiles; tile += gridDim.x) {
        if (n_lr_stages > 0) {
          ok = __all_sync(0xffffffffu, bounded_wait<64>(bar_tmem_empty + 8 * tm.slot, tm.parity ^ 1u, env, kErrMmaWait));
          if (ok) tc_fence_after_sync();
          for (int l = 0; ok && l < n_lr_stages; ++l) {
            ok = __all_sync(0xffffffffu, bounded_wait<64>(bar_op_full + 8 * op.slot, op.parity, env, kErrMmaWait));
            if (!ok) break;
            const uint32_t a = smem_base + op.slot * kOsStageBytes, b = a + kOpATile;
            if (issuer) {
#pragma unroll
              for (int kk = 0; kk < 4; ++kk) {
                umma_f16(tmem_base + tm.slot * 2 * kBN, umma_desc_k_sw128(a, 32 * kk), umma_desc_k_sw128(b, 32 * kk), idesc_bf16,
                         (l > 0 || kk > 0) ? 1u : 0u);
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
          ok = __all_sync(0xffffffffu, bounded_wait<64>(bar_op_full + 8 * op.slot, op.parity, env, kErrMmaWait));
          if (!ok) break;
          const uint32_t a = smem_base + op.slot * kOsStageBytes, b = a + kOpATile;
          const int groups = (2 * st + 1 < G) ? 2 : 1;
          for (int v = 0; v < groups; ++v) {
            ok = __all_sync(0xffffffffu, bounded_wait<64>(bar_tmem_empty + 8 * tm.slot, tm.parity ^ 1u, env, kErrMmaWait));
            if (!ok) break;
            tc_fence_after_sync();
            const uint32_t d = tmem_base + tm.slot * 2 * kBN;
            if (issuer) {
              // bytes [64 v, 64 v + 64) of every code row: group v of the stage, two MMAs of K = 32
              umma_f8(d, umma_desc_k_sw128(a, 64 * v), umma_desc_k_sw128(b, 64 * v), idesc_f8, 0u);
              umma_f8(d, umma_desc_k_sw128(a, 64 * v + 32), umma_desc_k_sw128(b, 64 * v + 32), idesc_f8, 1u);
              umma_commit(bar_tmem_full + 8 * tm.slot);
            }
            tm.advance();
          }
          if (!ok) break;
          if (issuer) umma_commit(bar_op_empty + 8 * op.slot);
          op.advance();
        }
      }
    } else if (live && warp == 3) {
      // ------------------------------------------------------------------ scale-MMA issuer
      // The outer products S_g come from a second issuing warp: one thread needs some 40 cycles per tcgen05
      // instruction, and with a group per TMEM slot the issue time sits on the hand-over path.  Both warps wait for
      // the same barriers and both commit: op_empty and tmem_full count two arrivals.
      constexpr uint32_t idesc_bf16 = umma_idesc(1, 1, kBM, kBN);
      const bool issuer = elect_one_lane();
      Ring<kOsStages> op;
      Ring<kTmemSlots> tm;
      bool ok = true;
      for (int tile = blockIdx.x; ok && tile < num_tiles; tile += gridDim.x) {
        if (n_lr_stages > 0) {   // nothing to add to the low-rank slot: sign off in step with the other warp
          ok = __all_sync(0xffffffffu, bounded_wait<64>(bar_tmem_empty + 8 * tm.slot, tm.parity ^ 1u, env, kErrMmaWait));
          for (int l = 0; ok && l < n_lr_stages; ++l) {
            ok = __all_sync(0xffffffffu, bounded_wait<64>(bar_op_full + 8 * op.slot, op.parity, env, kErrMmaWait));
            if (!ok) break;
            if (issuer) mbar_arrive(bar_op_empty + 8 * op.slot);
            op.advance();
          }
          if (!ok) break;
          if (issuer) mbar_arrive(bar_tmem_full + 8 * tm.slot);
          tm.advance();
        }
        for (int st = 0; ok && st < n_int_stages; ++st) {
          ok = __all_sync(0xffffffffu, bounded_wait<64>(bar_op_full + 8 * op.slot, op.parity, env, kErrMmaWait));
          if (!ok) break;
          const uint32_t sa = smem_base + op.slot * kOsStageBytes + kOpATile + kOpBTile, sb = sa + kOsSopTile;
          const int groups = (2 * st + 1 < G) ? 2 : 1;
          for (int v = 0; v < groups; ++v) {
            ok = __all_sync(0xffffffffu, bounded_wait<64>(bar_tmem_empty + 8 * tm.slot, tm.parity ^ 1u, env, kErrMmaWait));
            if (!ok) break;
            tc_fence_after_sync();
            if (issuer) {
              const uint32_t ca = sa + 128 * v, cb = sb + 128 * v;   // this group's chunk of every row group
              umma_f16(tmem_base + tm.slot * 2 * kBN + kBN, sop_desc(ca, zero_base - ca), sop_desc(cb, zero_base - cb), idesc_bf16, 0u);
              umma_commit(bar_tmem_full + 8 * tm.slot);
            }
            tm.advance();
          }
          if (!ok) break;
          if (issuer) umma_commit(bar_op_empty + 8 * op.slot);
          op.advance();
        }
      }
    }
  } else {
    set_max_regs_inc<kRegsEpilogue>();
    if (live) {
      // ------------------------------------------------------------------ epilogue warps
      // Warp ew owns TMEM lanes 32 * (ew % 4) .. +31 (token rows) and the 32-column block ew / 4; a thread owns one
      // row and the block's 32 output channels.  Per group two fragments of 16 columns, each a pair of TMEM loads
      // (P and S) and eight packed multiply-adds; the four warps of a scheduler hide one another's TMEM latency.
      const int ew = warp - kEpiWarp0;
      const int quarter = ew & 3, colblk = ew >> 2;
      const uint32_t t_lane = tmem_base + (static_cast<uint32_t>(32 * quarter) << 16) + kEpiCols * colblk;
      Ring<kTmemSlots> tm;
      bool ok = true;
      for (int tile = blockIdx.x; ok && tile < num_tiles; tile += gridDim.x) {
        const int m0 = (tile / p.tiles_n) * kBM, n0 = (tile % p.tiles_n) * kBN;
        const int row = m0 + 32 * quarter + lane;
        const int ch0 = n0 + kEpiCols * colblk;
        const bool dbg_tile = DEBUG && p.dbg_P != nullptr && m0 == p.dbg_m0 && n0 == p.dbg_n0;
        float2 acc[16];  // pair k: channels ch0 + 2 k, ch0 + 2 k + 1
        ok = __all_sync(0xffffffffu, bounded_wait(bar_tmem_full + 8 * tm.slot, tm.parity, env, kErrEpilogueWait));
        if (!ok) break;
        tc_fence_after_sync();
        if (n_lr_stages > 0) {
          // The low-rank product T L2 (FP32) seeds the accumulators.
          const uint32_t t = t_lane + tm.slot * 2 * kBN;
          uint32_t lo[16], hi[16];
          tmem_ld_32x32b_x16(t, lo);
          tmem_ld_32x32b_x16(t + 16, hi);
          tmem_wait_ld_into(lo, hi);
          tc_fence_before_sync();
          __syncwarp();
          if (lane == 0) mbar_arrive(bar_tmem_empty + 8 * tm.slot);
          tm.advance();
#pragma unroll
          for (int k = 0; k < 8; ++k) {
            acc[k] = make_float2(__uint_as_float(lo[2 * k]), __uint_as_float(lo[2 * k + 1]));
            acc[8 + k] = make_float2(__uint_as_float(hi[2 * k]), __uint_as_float(hi[2 * k + 1]));
          }
          ok = __all_sync(0xffffffffu, bounded_wait(bar_tmem_full + 8 * tm.slot, tm.parity, env, kErrEpilogueWait));
          if (!ok) break;
          tc_fence_after_sync();
        } else {
#pragma unroll
          for (int j = 0; j < 16; ++j) acc[j] = make_float2(0.0f, 0.0f);
        }
        // Invariant at the top of each iteration: the group's slot has been waited for.
        for (int g = 0; g < G; ++g) {
          const uint32_t t = t_lane + tm.slot * 2 * kBN;
          int32_t* d0 = nullptr;
          if (DEBUG) {
            if (dbg_tile) d0 = p.dbg_P + (static_cast<size_t>(32 * quarter + lane) * G + g) * kBN + kEpiCols * colblk;
          }
          uint32_t pv[16], sv[16];
          tmem_ld_32x32b_x16(t, pv);
          tmem_ld_32x32b_x16(t + kBN, sv);
          tmem_wait_ld_into(pv, sv);
          fma_fragment<DEBUG>(pv, sv, acc, d0);
          tmem_ld_32x32b_x16(t + 16, pv);
          tmem_ld_32x32b_x16(t + kBN + 16, sv);
          tmem_wait_ld_into(pv, sv);
          // The whole slot is in registers: hand it back to the MMA warp.
          tc_fence_before_sync();
          __syncwarp();
          if (lane == 0) mbar_arrive(bar_tmem_empty + 8 * tm.slot);
          tm.advance();
          fma_fragment<DEBUG>(pv, sv, acc + 8, DEBUG && d0 ? d0 + 16 : nullptr);
          if (g + 1 < G) {
            ok = __all_sync(0xffffffffu, bounded_wait(bar_tmem_full + 8 * tm.slot, tm.parity, env, kErrEpilogueWait));
            if (!ok) break;
            tc_fence_after_sync();
          }
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
