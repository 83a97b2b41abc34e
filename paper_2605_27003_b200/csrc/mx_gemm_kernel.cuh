// Kernel 2 of the MXFP4 variant: block-scaled FP4 GEMM + low-rank up-projection + bias + BF16 store.
//
//   Y[m,n] = sum_b 2^(ea[m,b]-127) 2^(ew[b,n]-127) sum_{k in block b} a[m,k] w[k,n]  +  sum_j T[m,j] L2[j,n]  +  b[n]
//
// a, w are E2M1 elements, ea / ew the E8M0 exponents of their 32-element blocks along K (OCP MX v1.0, the data
// format the paper's Table 1 names).  tcgen05.mma kind::mxf4.block_scale applies both block scales inside the
// tensor core and accumulates in FP32, so -- unlike the INT4 kernel -- nothing is rescaled on the CUDA cores and
// the whole K extent accumulates into one TMEM tile; the epilogue runs once per output tile.
//
// Three kernels in this file: mx_gemm_kernel (one CTA per 128 x 256 tile; described next), mx_gemm2_kernel<false>
// (the default: a cluster of two CTAs per 256 x 256 tile, tcgen05 cta_group::2) and mx_gemm2_kernel<true> (the same
// with an epilogue that, instead of storing Y, quantizes it for the next layer); the latter two are described in
// front of their definition.
//
// Persistent kernel, one CTA per SM, 128 x 256 output tiles, column tile fastest.  At the FP4 rate the tensor
// core consumes operands faster than L2 and the shared-memory port deliver them, so the tile is as wide as TMEM
// allows (operand bytes per MAC fall by a quarter against 128 x 128).  Warp roles:
//   warp 0      producer (all lanes loop, one elected lane issues): per stage of 256 K elements one TMA each for the packed A tile (128 rows x
//               128 bytes) and B tile (256 rows x 128 bytes), 128-byte swizzle, and bulk copies for their scale
//               bytes (1 KiB per 128 rows: two 512-byte atoms, the layout the tensor core wants); the BF16
//               low-rank operands T and L2 go through the same ring first.
//   warp 1      MMA issuer (all lanes loop, one elected lane issues): per stage six tcgen05.cp (scale atoms, shared memory -> TMEM: 32 lanes x
//               128 bits, replicated to the four lane quarters) and four tcgen05.mma kind::mxf4 (128 x 256, K = 64
//               each: two scale blocks per row, selected by the scale-factor id 0 / 2 inside the 4-byte TMEM
//               column); kind::f16 for [T_hi | T_lo] [L2 | L2]^T into the same accumulator first.  tcgen05.cp
//               and tcgen05.mma of one thread execute in issue order, so one TMEM scale region serves every stage.
//   warp 2      TMEM allocation / release.
//   warps 4-19  epilogue: TMEM (32x32b loads, a token row per thread, 64 columns per warp) + bias -> BF16 ->
//               global.  One accumulator (256 columns) plus the scale columns fill TMEM, so the MMA warp waits
//               for the epilogue to drain it before the next tile: sixteen warps pull the whole accumulator into
//               registers at once and hand it back before they convert and store.
//
// Every wait is bounded (pipeline.cuh).
#pragma once

#include <cuda_bf16.h>
#include <stdint.h>

#include "pipeline.cuh"
#include "ptx.cuh"
#include "quantize_kernel.cuh"

namespace w4a4 {

constexpr int kMxBN = 256;                       // output tile columns
constexpr int kMxBK = 256;                       // K elements per stage = 128 bytes per operand row
constexpr int kMxStages = 4;
constexpr int kMxThreads = 640;
constexpr int kMxEpiWarp0 = 4, kMxEpiWarps = 16;
constexpr uint32_t kMxATile = kBM * 128;         // 16 KiB
constexpr uint32_t kMxBTile = kMxBN * 128;       // 32 KiB
constexpr uint32_t kMxSfTile = 2 * 512;          // scale bytes of 128 rows x 8 blocks: two atoms
constexpr uint32_t kMxStageBytes = kMxATile + kMxBTile + 3 * kMxSfTile;   // A, B, scales of A and of both halves of B
constexpr uint32_t kMxNumBarriers = 2 * kMxStages + 2;
constexpr uint32_t kMxSmemBytes = 1024 + kMxStages * kMxStageBytes + kMxNumBarriers * 8 + 16;
constexpr uint32_t kMxTmemSfA = 256, kMxTmemSfB = 264;   // columns: accumulator 0..255, then 8 + 16 scale columns
static_assert(kBM == 128, "the scale-factor atoms and the TMEM layout assume 128-row tiles");
static_assert(kMxStageBytes % 1024 == 0, "operand tiles must stay 1024-byte aligned");

struct MxGemmParams {
  const float* bias;     // [N] or nullptr
  uint16_t* Y;           // [M, N] BF16
  const uint8_t* sfa;    // activation scale atoms: [ceil(M/128)][K/128][512]
  const uint8_t* sfb;    // weight scale atoms:     [N/128][K/128][512]
  int M, N, K, r;
  int tiles_m, tiles_n;
  int* err;
  // Clip-ratio search (Eq. 10): when yref is set, Y is not stored; the squared distance between the layer's
  // BF16 output and yref is accumulated into *sq_err instead.
  const uint16_t* yref;  // [M, N] BF16 or nullptr
  double* sq_err;
  int act;              // output activation: 0 none, 1 GELU (tanh form)
  int run;              // CTA-pair kernel: consecutive column tiles of a row pair that one cluster takes at a time
};

// One lane of a converged warp.  The MMA warp runs its loop with all lanes (waits included) and only predicates
// the tcgen05 instructions on this: everything they take as operands then stays warp-uniform for the compiler,
// which keeps descriptors and addresses in uniform registers instead of converting them per instruction
// (elect_one_lane() comes from pipeline.cuh).

// Shared-memory descriptor of one scale atom (32 rows x 16 bytes, rows contiguous): K-major, no swizzle, 8-row
// core matrices 128 bytes apart.
__device__ __forceinline__ uint64_t mx_sf_desc(uint32_t smem_addr) {
  uint64_t d = 0;
  d |= static_cast<uint64_t>((smem_addr >> 4) & 0x3FFFu);
  d |= static_cast<uint64_t>(1u) << 16;
  d |= static_cast<uint64_t>((128u >> 4) & 0x3FFFu) << 32;
  d |= static_cast<uint64_t>(1u) << 46;
  return d;
}
__device__ __forceinline__ void tmem_cp_32x128b_warpx4(uint32_t taddr, uint64_t sdesc) {
  asm volatile("tcgen05.cp.cta_group::1.32x128b.warpx4 [%0], %1;" ::"r"(taddr), "l"(sdesc) : "memory");
}
// Instruction descriptor of kind::mxf4 (block-scaled): E2M1 x E2M1, E8M0 scales, K-major operands, K = 64.
__host__ __device__ constexpr uint32_t mx_idesc(uint32_t M, uint32_t N, uint32_t a_sf_id, uint32_t b_sf_id) {
  return (b_sf_id << 4) | (1u << 7) | (1u << 10) | ((N >> 3) << 17) | (1u << 23) | ((M >> 4) << 24) | (a_sf_id << 29);
}
__device__ __forceinline__ void umma_mxf4(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t tsfa,
                                          uint32_t tsfb, uint32_t accumulate) {
  asm volatile(
      "{\n"
      ".reg .pred p;\n"
      "setp.ne.b32 p, %4, 0;\n"
      "tcgen05.mma.cta_group::1.kind::mxf4.block_scale.block32 [%0], %1, %2, %3, [%5], [%6], p;\n"
      "}\n" ::"r"(d_tmem),
      "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate), "r"(tsfa), "r"(tsfb)
      : "memory");
}
// Plain (untiled) bulk copy global -> shared, completion on an mbarrier.  Both addresses 16-byte aligned,
// size a multiple of 16.
__device__ __forceinline__ void bulk_load(uint32_t dst_smem, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst_smem),
               "l"(src), "r"(bytes), "r"(bar)
               : "memory");
}

__global__ void __launch_bounds__(kMxThreads, 1)
mx_gemm_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
               const __grid_constant__ CUtensorMap tmT, const __grid_constant__ CUtensorMap tmL2, const MxGemmParams p) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* smem = smem_raw + (smem_base - smem_u32(smem_raw));
  const uint32_t bar_base = smem_base + kMxStages * kMxStageBytes;
  const uint32_t bar_full = bar_base;
  const uint32_t bar_empty = bar_full + 8 * kMxStages;
  const uint32_t bar_acc_full = bar_empty + 8 * kMxStages;
  const uint32_t bar_acc_empty = bar_acc_full + 8;
  const uint32_t misc_off = (bar_acc_empty + 8) - smem_base;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + misc_off);
  volatile int* s_abort = reinterpret_cast<volatile int*>(smem + misc_off + 4);

  const int warp = __shfl_sync(0xffffffffu, static_cast<int>(threadIdx.x >> 5), 0), lane = threadIdx.x & 31;  // provably warp-uniform
  const int n_k_stages = p.K / kMxBK;
  const int n_lr_stages = p.r > 0 ? (2 * p.r + 63) / 64 : 0;
  const int atoms_k = p.K / 128;
  const int num_tiles = p.tiles_m * p.tiles_n;
  const WaitEnv env{p.err, s_abort, kWaitLimitNs};

  if (threadIdx.x == 0) {
    *s_abort = (*reinterpret_cast<volatile int*>(p.err) != 0) ? 1 : 0;
    for (int i = 0; i < kMxStages; ++i) {
      mbar_init(bar_full + 8 * i, 1);
      mbar_init(bar_empty + 8 * i, 1);
    }
    mbar_init(bar_acc_full, 1);
    mbar_init(bar_acc_empty, kMxEpiWarps);
    mbar_fence_init();
    fence_proxy_async_smem();
    tma_prefetch_desc(&tmA);
    tma_prefetch_desc(&tmB);
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

  // Shared-memory stage: A tile | B tile (256 rows) | scale atoms of A | of B rows 0..127 | of B rows 128..255.
  if (live && warp == 0) {
    // ------------------------------------------------------------------ producer (all lanes loop, one issues)
    const bool issuer = elect_one_lane();
    Ring<kMxStages> rg;
    bool ok = true;
    for (int tile = blockIdx.x; ok && tile < num_tiles; tile += gridDim.x) {
      const int tm = tile / p.tiles_n, tn = tile % p.tiles_n;
      const int m0 = tm * kBM, n0 = tn * kMxBN;
      const bool upper = n0 + 128 < p.N;  // does the tile's second 128-column half exist?
      for (int st = 0; st < n_lr_stages + n_k_stages; ++st) {
        ok = __all_sync(0xffffffffu, bounded_wait<128>(bar_empty + 8 * rg.slot, rg.parity ^ 1u, env, kErrProducerWait));
        if (!ok) break;
        const uint32_t full = bar_full + 8 * rg.slot;
        const uint32_t dst = smem_base + rg.slot * kMxStageBytes;
        if (st < n_lr_stages) {
          if (issuer) {
            mbar_arrive_expect_tx(full, kMxATile + kMxBTile);
            tma_load_2d(dst, &tmT, full, st * 64, m0);
            tma_load_2d(dst + kMxATile, &tmL2, full, st * 64, n0);  // rows past N arrive as zeros
          }
        } else if (issuer) {
          const int ks = st - n_lr_stages;
          const uint32_t sf = dst + kMxATile + kMxBTile;
          mbar_arrive_expect_tx(full, kMxATile + kMxBTile + (upper ? 3u : 2u) * kMxSfTile);
          tma_load_2d(dst, &tmA, full, ks * 128, m0);
          tma_load_2d(dst + kMxATile, &tmB, full, ks * 128, n0);
          bulk_load(sf, p.sfa + (static_cast<size_t>(tm) * atoms_k + 2 * ks) * 512, kMxSfTile, full);
          bulk_load(sf + kMxSfTile, p.sfb + (static_cast<size_t>(2 * tn) * atoms_k + 2 * ks) * 512, kMxSfTile, full);
          if (upper)
            bulk_load(sf + 2 * kMxSfTile, p.sfb + (static_cast<size_t>(2 * tn + 1) * atoms_k + 2 * ks) * 512, kMxSfTile, full);
        }
        rg.advance();
      }
    }
  } else if (live && warp == 1) {
    // ------------------------------------------------------------------ MMA issuer (all lanes loop, one issues)
    constexpr uint32_t idesc_bf16 = umma_idesc(1, 1, kBM, kMxBN);
    const bool issuer = elect_one_lane();
    Ring<kMxStages> rg;
    Ring<1> ab;
    bool ok = true;
    for (int tile = blockIdx.x; ok && tile < num_tiles; tile += gridDim.x) {
      ok = __all_sync(0xffffffffu, bounded_wait<64>(bar_acc_empty, ab.parity ^ 1u, env, kErrMmaWait));
      if (!ok) break;
      tc_fence_after_sync();
      const uint32_t d = tmem_base;
      uint32_t accumulate = 0;
      for (int st = 0; ok && st < n_lr_stages + n_k_stages; ++st) {
        ok = __all_sync(0xffffffffu, bounded_wait<64>(bar_full + 8 * rg.slot, rg.parity, env, kErrMmaWait));
        if (!ok) break;
        const uint32_t a = smem_base + rg.slot * kMxStageBytes, b = a + kMxATile;
        if (st < n_lr_stages) {
          if (issuer) {
#pragma unroll
            for (int kk = 0; kk < 4; ++kk)
              umma_f16(d, umma_desc_k_sw128(a, 32 * kk), umma_desc_k_sw128(b, 32 * kk), idesc_bf16, kk > 0 ? 1u : accumulate);
          }
        } else if (issuer) {
          // TMEM scale columns: A: 4 per K atom (one per 32 rows); B: 8 per K atom (256 rows).  The columns of
          // a missing upper half keep whatever they held: they scale zero operands into columns never stored.
          const uint32_t sf = b + kMxBTile;
#pragma unroll
          for (int t = 0; t < 2; ++t) {
            tmem_cp_32x128b_warpx4(tmem_base + kMxTmemSfA + 4 * t, mx_sf_desc(sf + 512 * t));
            tmem_cp_32x128b_warpx4(tmem_base + kMxTmemSfB + 8 * t, mx_sf_desc(sf + kMxSfTile + 512 * t));
            tmem_cp_32x128b_warpx4(tmem_base + kMxTmemSfB + 8 * t + 4, mx_sf_desc(sf + 2 * kMxSfTile + 512 * t));
          }
#pragma unroll
          for (int j = 0; j < 4; ++j) {  // bytes [32 j, 32 j + 32) of every row: scale blocks 2 j, 2 j + 1
            const uint32_t id = 2u * (j & 1);
            umma_mxf4(d, umma_desc_k_sw128(a, 32 * j), umma_desc_k_sw128(b, 32 * j), mx_idesc(kBM, kMxBN, id, id),
                      (tmem_base + kMxTmemSfA + 4 * (j >> 1)) | (id << 30), (tmem_base + kMxTmemSfB + 8 * (j >> 1)) | (id << 30),
                      j > 0 ? 1u : accumulate);
          }
        }
        accumulate = 1;
        if (issuer) umma_commit(bar_empty + 8 * rg.slot);
        rg.advance();
      }
      if (!ok) break;
      if (issuer) umma_commit(bar_acc_full);
      ab.advance();
    }
  } else if (live && warp >= kMxEpiWarp0) {
    // ------------------------------------------------------------------ epilogue
    // Warp ew: TMEM lanes 32 * (ew % 4) .. + 31 (token rows), columns 64 * (ew / 4) .. + 63.  The buffer goes back to
    // the MMA warp as soon as the warp's part of it is in registers, before it is converted and stored.
    const int ew = warp - kMxEpiWarp0;
    const int quarter = ew & 3, colblk = ew >> 2;
    Ring<1> ab;
    bool ok = true;
    for (int tile = blockIdx.x; ok && tile < num_tiles; tile += gridDim.x) {
      const int m0 = (tile / p.tiles_n) * kBM, n0 = (tile % p.tiles_n) * kMxBN;
      const int row = m0 + 32 * quarter + lane;
      ok = bounded_wait(bar_acc_full, ab.parity, env, kErrEpilogueWait);
      if (!ok) break;
      tc_fence_after_sync();
      const uint32_t t_row = tmem_base + (static_cast<uint32_t>(32 * quarter) << 16) + 64 * colblk;
      uint32_t v[4][16];
#pragma unroll
      for (int c = 0; c < 4; ++c) tmem_ld_32x32b_x16(t_row + 16 * c, v[c]);
      tmem_wait_ld();
      tc_fence_before_sync();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar_acc_empty);
      const int ch0 = n0 + 64 * colblk;
      if (p.yref != nullptr) {
        // Eq. 10's objective over this thread's 64 outputs, Y_hat rounded to BF16 as the forward stores it.
        float e = 0.0f;
        if (row < p.M && ch0 < p.N) {
          const uint4* yr = reinterpret_cast<const uint4*>(p.yref + static_cast<size_t>(row) * p.N + ch0);
#pragma unroll
          for (int c = 0; c < 4; ++c) {
#pragma unroll
            for (int h = 0; h < 2; ++h) {
              const uint4 ref = __ldg(yr + 2 * c + h);
              const uint32_t rw[4] = {ref.x, ref.y, ref.z, ref.w};
#pragma unroll
              for (int i = 0; i < 8; ++i) {
                const int col = 8 * h + i;
                const float b = p.bias ? __ldg(p.bias + ch0 + 16 * c + col) : 0.0f;
                const float y_hat = __bfloat162float(__float2bfloat16_rn(apply_activation(__uint_as_float(v[c][col]) + b, p.act)));
                const float y_ref = __uint_as_float((i & 1) ? (rw[i >> 1] & 0xffff0000u) : (rw[i >> 1] << 16));
                const float d = y_ref - y_hat;
                e = fmaf(d, d, e);
              }
            }
          }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) e += __shfl_xor_sync(0xffffffffu, e, o);
        if (lane == 0) atomicAdd(p.sq_err, static_cast<double>(e));
      } else if (row < p.M && ch0 < p.N) {
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          const int ch = ch0 + 16 * c;
          uint4 o[2];
          uint32_t* ow = reinterpret_cast<uint32_t*>(o);
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            const float4 b4 = p.bias ? __ldg(reinterpret_cast<const float4*>(p.bias + ch) + i) : make_float4(0.f, 0.f, 0.f, 0.f);
            float y0 = __uint_as_float(v[c][4 * i]) + b4.x, y1 = __uint_as_float(v[c][4 * i + 1]) + b4.y;
            float y2 = __uint_as_float(v[c][4 * i + 2]) + b4.z, y3 = __uint_as_float(v[c][4 * i + 3]) + b4.w;
            if (p.act != 0) {  // uniform over the grid: the plain layer pays one predicate per four outputs
              y0 = apply_activation(y0, p.act);
              y1 = apply_activation(y1, p.act);
              y2 = apply_activation(y2, p.act);
              y3 = apply_activation(y3, p.act);
            }
            __nv_bfloat162 lo = __floats2bfloat162_rn(y0, y1);
            __nv_bfloat162 hi = __floats2bfloat162_rn(y2, y3);
            ow[2 * i] = *reinterpret_cast<uint32_t*>(&lo);
            ow[2 * i + 1] = *reinterpret_cast<uint32_t*>(&hi);
          }
          uint4* y = reinterpret_cast<uint4*>(p.Y + static_cast<size_t>(row) * p.N + ch);
          y[0] = o[0];
          y[1] = o[1];
        }
      }
      ab.advance();
    }
  }

  // ---------------------------------------------------------------------- common tail
  tc_fence_before_sync();
  __syncthreads();
  if (*s_abort) {
    const uint64_t t0 = global_timer_ns();
    while (global_timer_ns() - t0 < 200000ull) __nanosleep(1000);
    __syncthreads();
  }
  if (warp == 2) {
    tc_fence_after_sync();
    tmem_dealloc(tmem_base, 512);
  }
}

// ---------------------------------------------------------------------------------------------------------------
// The same GEMM on pairs of CTAs (a thread-block cluster of two, tcgen05 cta_group::2).  mx_gemm_kernel is bound
// by the bytes that come from L2 into shared memory.  With cta_group::2 one MMA spans both SMs of the pair: a
// 256 x 256 x 64 product whose A rows 0..127 / 128..255 and whose B rows (output columns) 0..127 / 128..255 lie in
// the shared memory of CTA 0 / CTA 1, at the same offsets, and whose accumulator rows land in the TMEM of the CTA
// that holds the A rows.  Each CTA therefore fetches its own A tile and only HALF of the B tile: 35 KB per stage
// instead of 51 KB for the same 128 x 256 outputs per CTA, and the ring is six stages deep instead of four.
//
// CTA 0 (the leader) issues every tcgen05.cp and tcgen05.mma for the pair.  Cross-CTA signalling:
//   full[s]    (leader)   both CTAs' TMA loads of stage s report their bytes here (cta_group::2 loads may name a
//                         barrier of the neighbour); the leader's producer posts the expected total;
//   empty[s]   (both)     the leader commits its MMAs onto its own barrier and onto the neighbour's;
//   acc_full   (both)     likewise;
//   acc_empty  (leader)   all 32 epilogue warps of the pair have pulled their part of the accumulator.
// Scale factors: every CTA needs the A scales of its own rows and the B scales of all 256 columns in its own TMEM;
// tcgen05.cp.cta_group::2 copies them from each CTA's own shared memory.
__device__ __forceinline__ void tmem_cp2_32x128b_warpx4(uint32_t taddr, uint64_t sdesc) {
  asm volatile("tcgen05.cp.cta_group::2.32x128b.warpx4 [%0], %1;" ::"r"(taddr), "l"(sdesc) : "memory");
}
__device__ __forceinline__ void umma2_mxf4(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t tsfa,
                                           uint32_t tsfb, uint32_t accumulate) {
  asm volatile(
      "{\n"
      ".reg .pred p;\n"
      "setp.ne.b32 p, %4, 0;\n"
      "tcgen05.mma.cta_group::2.kind::mxf4.block_scale.block32 [%0], %1, %2, %3, [%5], [%6], p;\n"
      "}\n" ::"r"(d_tmem),
      "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate), "r"(tsfa), "r"(tsfb)
      : "memory");
}
constexpr int kMx2Stages = 6;
constexpr uint32_t kMx2BHalf = kMxBTile / 2;                                  // 16 KiB: this CTA's 128 rows of B
constexpr uint32_t kMx2StageBytes = kMxATile + kMx2BHalf + 3 * kMxSfTile;      // 35 KiB
constexpr uint32_t kMx2NumBarriers = 2 * kMx2Stages + 2;
constexpr uint32_t kMx2SmemBytes = 1024 + kMx2Stages * kMx2StageBytes + kMx2NumBarriers * 8 + 16;
static_assert(kMx2StageBytes % 1024 == 0, "operand tiles must stay 1024-byte aligned");

// ---- Fused form (FUSE = true): the epilogue does not store the layer's output but quantizes it for the NEXT layer
// (Sec. III: the FFN's second linear reads GELU of the first): y -> BF16 -> x_hat = y / lambda' -> MXFP4 codes and
// block exponents straight into the next layer's workspace, exactly what kernel 1 would produce from the stored
// output, and the next layer's low-rank projection T' = bf16(x_hat) L1' (Eq. 7) on the tensor core: the epilogue
// leaves bf16(x_hat) of the tile in shared memory as a K-major operand, a fourth control warp multiplies it by the
// matching 256 rows of L1' (tcgen05.mma kind::f16, M = 256 over the pair, N = r') into a small TMEM accumulator
// that stays resident while the cluster walks a run of column tiles of one row pair (work is dealt to clusters in
// such runs), and is added into an FP32 [M, r'] array when the run ends.
// Shared memory: four stages instead of six, the 64 KiB x_hat tile, 16 KiB for the L1' tile (four K slices of
// r'/2 rows, packed at whole swizzle atoms; for r' <= 32 they fill the lower half and the upper half holds one
// 512-byte table per epilogue warp: the bias and the next layer's 1/lambda of the warp's 64 channels).
// Barriers: xh_full (leader; 32 epilogue warps: "x_hat tile written"), xh_empty (both; committed after the T MMAs:
// x_hat and L1' tiles may be overwritten), l1_full (leader; TMA bytes of both CTAs' L1' halves), t_full[2] (both;
// committed after the last T MMA of a row pair), t_empty[2] (leader; 8 warps: "T buffer read").
constexpr int kMx2FuseStages = 4;
constexpr uint32_t kMx2XhBytes = 4 * kMxATile;       // 128 rows x 256 channels BF16: four K slices of 64 channels
constexpr uint32_t kMx2L1SliceBytes = 4096;           // up to 32 rows (r' / 2 <= 32) x 128 bytes
constexpr uint32_t kMx2FuseBarriers = 2 * kMx2FuseStages + 2 + 7;
constexpr uint32_t kMx2FuseSmemBytes = 1024 + kMx2FuseStages * kMx2StageBytes + kMx2XhBytes + 4 * kMx2L1SliceBytes +
                                       kMx2FuseBarriers * 8 + 16;
static_assert(kMx2FuseSmemBytes <= 232448, "shared memory budget of one CTA");
constexpr uint32_t kMxTmemT = 320;                    // two T buffers of 64 columns: 320..447

struct MxNextParams {
  const float* rlam;     // next layer's reciprocal smoothing factors [N]
  const float* rho;      // the next layer's clip ratio (one float on the device)
  uint8_t* codes;        // next layer's packed E2M1 codes [M, N/2]
  uint8_t* sfa;          // next layer's activation scale atoms [ceil(M/128)][N/128][512]
  float* t32;            // next layer's T accumulators [M, r2] FP32, zero before the launch
  int r2;                // next layer's rank: 0, 16, 32 or 64
};

// MXFP4 conversion of 32 consecutive channels held by one thread (the same arithmetic as kernel 1's
// mxfp4_block16, without the shuffle): returns the E8M0 exponent byte, packed codes in w[0..3].
__device__ __forceinline__ uint32_t mxfp4_block32(const uint32_t (&lo)[16], const uint32_t (&hi)[16], float rho, uint4& w) {
  float a0 = 0.0f, a1 = 0.0f;
#pragma unroll
  for (int e = 0; e < 16; e += 2) {
    a0 = fmaxf(a0, fmaxf(fabsf(__uint_as_float(lo[e])), fabsf(__uint_as_float(hi[e]))));
    a1 = fmaxf(a1, fmaxf(fabsf(__uint_as_float(lo[e + 1])), fabsf(__uint_as_float(hi[e + 1]))));
  }
  const float a = fmaxf(a0, a1);
  const uint32_t field = (__float_as_uint(__fmul_rn(rho, a)) >> 23) & 0xffu;
  const uint32_t ex = field > 2u ? field - 2u : 0u;
  const float inv = __uint_as_float((254u - ex) << 23);
  float t[8];
#pragma unroll
  for (int e = 0; e < 8; ++e) t[e] = __fmul_rn(__uint_as_float(lo[e]), inv);
  w.x = e2m1x8(t);
#pragma unroll
  for (int e = 0; e < 8; ++e) t[e] = __fmul_rn(__uint_as_float(lo[8 + e]), inv);
  w.y = e2m1x8(t);
#pragma unroll
  for (int e = 0; e < 8; ++e) t[e] = __fmul_rn(__uint_as_float(hi[e]), inv);
  w.z = e2m1x8(t);
#pragma unroll
  for (int e = 0; e < 8; ++e) t[e] = __fmul_rn(__uint_as_float(hi[8 + e]), inv);
  w.w = e2m1x8(t);
  return ex;
}

template <bool FUSE>
__global__ void __launch_bounds__(kMxThreads, 1)
mx_gemm2_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmBhalf,
                const __grid_constant__ CUtensorMap tmT, const __grid_constant__ CUtensorMap tmL2half,
                const __grid_constant__ CUtensorMap tmSFA, const __grid_constant__ CUtensorMap tmSFB,
                const __grid_constant__ CUtensorMap tmL1T, const MxGemmParams p, const MxNextParams nx) {
  constexpr int STAGES = FUSE ? kMx2FuseStages : kMx2Stages;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* smem = smem_raw + (smem_base - smem_u32(smem_raw));
  const uint32_t xh_base = smem_base + STAGES * kMx2StageBytes;          // FUSE only: x_hat tile, then the L1' tile
  const uint32_t l1_base = xh_base + kMx2XhBytes;
  const uint32_t bar_base = FUSE ? l1_base + 4 * kMx2L1SliceBytes : xh_base;
  const uint32_t bar_full = bar_base;
  const uint32_t bar_empty = bar_full + 8 * STAGES;
  const uint32_t bar_acc_full = bar_empty + 8 * STAGES;
  const uint32_t bar_acc_empty = bar_acc_full + 8;
  const uint32_t bar_xh_full = bar_acc_empty + 8;      // the next seven exist only when FUSE
  const uint32_t bar_xh_empty = bar_xh_full + 8;
  const uint32_t bar_l1_full = bar_xh_empty + 8;
  const uint32_t bar_t_full = bar_l1_full + 8;          // [2]
  const uint32_t bar_t_empty = bar_t_full + 16;         // [2]
  const uint32_t misc_off = (FUSE ? bar_t_empty + 16 : bar_acc_empty + 8) - smem_base;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + misc_off);
  volatile int* s_abort = reinterpret_cast<volatile int*>(smem + misc_off + 4);

  const int warp = __shfl_sync(0xffffffffu, static_cast<int>(threadIdx.x >> 5), 0), lane = threadIdx.x & 31;  // provably warp-uniform
  const uint32_t rank = cluster_ctarank();
  const bool leader = rank == 0;
  const int n_k_stages = p.K / kMxBK;
  const int n_lr_stages = p.r > 0 ? (2 * p.r + 63) / 64 : 0;
  // Work is dealt to the clusters in runs of p.run consecutive column tiles of one row pair (run = 1: plain
  // interleaving).  The fused form uses longer runs so that the next layer's T can stay in TMEM over a run; short
  // enough that the clusters running at the same time still share their A rows in L2.
  const int run = p.run;
  const int runs_per_pair = (p.tiles_n + run - 1) / run;
  const int num_runs = ((p.tiles_m + 1) / 2) * runs_per_pair;
  const int cluster_id = blockIdx.x >> 1, num_clusters = gridDim.x >> 1;
  const WaitEnv env{p.err, s_abort, kWaitLimitNs};
  if (threadIdx.x == 0) {
    *s_abort = (*reinterpret_cast<volatile int*>(p.err) != 0) ? 1 : 0;
    for (int i = 0; i < STAGES; ++i) {
      mbar_init(bar_full + 8 * i, 1);
      mbar_init(bar_empty + 8 * i, 1);
    }
    mbar_init(bar_acc_full, 1);
    mbar_init(bar_acc_empty, 2 * kMxEpiWarps);
    if (FUSE) {
      mbar_init(bar_xh_full, 2 * kMxEpiWarps);
      mbar_init(bar_xh_empty, 1);
      mbar_init(bar_l1_full, 1);
      for (int i = 0; i < 2; ++i) {
        mbar_init(bar_t_full + 8 * i, 1);
        mbar_init(bar_t_empty + 8 * i, 8);
      }
      tma_prefetch_desc(&tmL1T);
    }
    mbar_fence_init();
    fence_proxy_async_smem();
    tma_prefetch_desc(&tmA);
    tma_prefetch_desc(&tmBhalf);
    tma_prefetch_desc(&tmSFA);
    tma_prefetch_desc(&tmSFB);
    if (p.r > 0) {
      tma_prefetch_desc(&tmT);
      tma_prefetch_desc(&tmL2half);
    }
  }
  if (warp == 2) {
    tmem_alloc2(smem_u32(tmem_slot), 512);
    tc_fence_before_sync();
  }
  __syncthreads();
  cluster_sync_all();  // both CTAs' barriers and TMEM exist before anything crosses over
  tc_fence_after_sync();
  const uint32_t tmem_base = __shfl_sync(0xffffffffu, *tmem_slot, 0);
  const bool live = __all_sync(0xffffffffu, *s_abort == 0);

  // Shared-memory stage: A tile | this CTA's half of B | scale atoms of A | of B columns 0..127 | of B columns 128..255.
  if (live && warp == 0) {
    // ------------------------------------------------------------------ producer (both CTAs; all lanes loop, one issues)
    // Rows and columns past the matrices (an odd count of row tiles; N = 128 mod 256) are filled with zeros by the
    // TMA unit and still count their bytes, so every stage reports the same total.
    const bool issuer = elect_one_lane();
    const uint32_t full0 = map_to_cta(bar_full, 0);
    Ring<STAGES> rg;
    bool ok = true;
    for (int q = cluster_id; ok && q < num_runs; q += num_clusters)
    for (int tn = (q % runs_per_pair) * run, tn1 = min(tn + run, p.tiles_n); ok && tn < tn1; ++tn) {
      const int tm = 2 * (q / runs_per_pair) + static_cast<int>(rank);
      const int m0 = tm * kBM, n0 = tn * kMxBN;
      for (int st = 0; st < n_lr_stages + n_k_stages; ++st) {
        ok = __all_sync(0xffffffffu, bounded_wait<128>(bar_empty + 8 * rg.slot, rg.parity ^ 1u, env, kErrProducerWait));
        if (!ok) break;
        const uint32_t full = full0 + 8 * rg.slot;
        const uint32_t dst = smem_base + rg.slot * kMx2StageBytes;
        if (st < n_lr_stages) {
          if (issuer) {
            if (leader) mbar_arrive_expect_tx(bar_full + 8 * rg.slot, 2 * (kMxATile + kMx2BHalf));
            tma2_load_2d(dst, &tmT, full, st * 64, m0);
            tma2_load_2d(dst + kMxATile, &tmL2half, full, st * 64, n0 + 128 * static_cast<int>(rank));
          }
        } else if (issuer) {
          const int ks = st - n_lr_stages;
          const uint32_t sf = dst + kMxATile + kMx2BHalf;
          if (leader) mbar_arrive_expect_tx(bar_full + 8 * rg.slot, 2 * kMx2StageBytes);
          tma2_load_2d(dst, &tmA, full, ks * 128, m0);
          tma2_load_2d(dst + kMxATile, &tmBhalf, full, ks * 128, n0 + 128 * static_cast<int>(rank));
          tma2_load_2d(sf, &tmSFA, full, ks * 256, tm);
          tma2_load_2d(sf + kMxSfTile, &tmSFB, full, ks * 256, 2 * tn);
          tma2_load_2d(sf + 2 * kMxSfTile, &tmSFB, full, ks * 256, 2 * tn + 1);
        }
        rg.advance();
      }
    }
  } else if (live && warp == 1 && leader) {
    // ------------------------------------------------------------------ MMA issuer (CTA 0, for the pair)
    constexpr uint32_t idesc_bf16 = umma_idesc(1, 1, 2 * kBM, kMxBN);
    const bool issuer = elect_one_lane();
    const uint32_t peer_empty = map_to_cta(bar_empty, 1), peer_acc_full = map_to_cta(bar_acc_full, 1);
    Ring<STAGES> rg;
    Ring<1> ab;
    bool ok = true;
    for (int q = cluster_id; ok && q < num_runs; q += num_clusters)
    for (int tn = (q % runs_per_pair) * run, tn1 = min(tn + run, p.tiles_n); ok && tn < tn1; ++tn) {
      ok = __all_sync(0xffffffffu, bounded_wait<64>(bar_acc_empty, ab.parity ^ 1u, env, kErrMmaWait));
      if (!ok) break;
      tc_fence_after_sync();
      const uint32_t d = tmem_base;
      uint32_t accumulate = 0;
      for (int st = 0; ok && st < n_lr_stages + n_k_stages; ++st) {
        ok = __all_sync(0xffffffffu, bounded_wait<64>(bar_full + 8 * rg.slot, rg.parity, env, kErrMmaWait));
        if (!ok) break;
        const uint32_t a = smem_base + rg.slot * kMx2StageBytes, b = a + kMxATile;
        if (st < n_lr_stages) {
          if (issuer) {
#pragma unroll
            for (int kk = 0; kk < 4; ++kk)
              umma2_f16(d, umma_desc_k_sw128(a, 32 * kk), umma_desc_k_sw128(b, 32 * kk), idesc_bf16, kk > 0 ? 1u : accumulate);
          }
        } else if (issuer) {
          const uint32_t sf = b + kMx2BHalf;
#pragma unroll
          for (int t = 0; t < 2; ++t) {
            tmem_cp2_32x128b_warpx4(tmem_base + kMxTmemSfA + 4 * t, mx_sf_desc(sf + 512 * t));
            tmem_cp2_32x128b_warpx4(tmem_base + kMxTmemSfB + 8 * t, mx_sf_desc(sf + kMxSfTile + 512 * t));
            tmem_cp2_32x128b_warpx4(tmem_base + kMxTmemSfB + 8 * t + 4, mx_sf_desc(sf + 2 * kMxSfTile + 512 * t));
          }
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            const uint32_t id = 2u * (j & 1);
            umma2_mxf4(d, umma_desc_k_sw128(a, 32 * j), umma_desc_k_sw128(b, 32 * j), mx_idesc(2 * kBM, kMxBN, id, id),
                       (tmem_base + kMxTmemSfA + 4 * (j >> 1)) | (id << 30), (tmem_base + kMxTmemSfB + 8 * (j >> 1)) | (id << 30),
                       j > 0 ? 1u : accumulate);
          }
        }
        accumulate = 1;
        if (issuer) {
          umma2_commit(bar_empty + 8 * rg.slot);
          umma2_commit(peer_empty + 8 * rg.slot);
        }
        rg.advance();
      }
      if (!ok) break;
      if (issuer) {
        umma2_commit(bar_acc_full);
        umma2_commit(peer_acc_full);
      }
      ab.advance();
    }
  } else if (FUSE && live && warp == 3 && nx.r2 > 0) {
    // ------------------------------------------------------------------ next layer's T = bf16(x_hat) L1' (FUSE)
    // Both CTAs fetch their half of the L1' rows that match the item's 256 channels; CTA 0 issues the MMAs.
    const bool issuer = elect_one_lane();
    const uint32_t idesc_t = umma_idesc(1, 1, 2 * kBM, static_cast<uint32_t>(nx.r2));
    const uint32_t l1_full0 = map_to_cta(bar_l1_full, 0);
    const uint32_t peer_xh_empty = map_to_cta(bar_xh_empty, 1), peer_t_full = map_to_cta(bar_t_full, 1);
    const int l1_rows = nx.r2 / 2;
    const uint32_t l1_pitch = l1_rows * 128 < 1024 ? 1024u : static_cast<uint32_t>(l1_rows) * 128u;   // whole swizzle atoms
    uint32_t k = 0, tb = 0, uses0 = 0, uses1 = 0;
    bool ok = true;
    for (int q = cluster_id; ok && q < num_runs; q += num_clusters)
    for (int tn0 = (q % runs_per_pair) * run, tn = tn0, tn1 = min(tn0 + run, p.tiles_n); ok && tn < tn1; ++tn, ++k) {
      // The x_hat and L1' tiles are free once the T MMAs of the previous item have completed.
      ok = __all_sync(0xffffffffu, bounded_wait<64>(bar_xh_empty, (k & 1u) ^ 1u, env, kErrMmaWait));
      if (!ok) break;
      const int n0 = tn * kMxBN;
      if (issuer) {
        if (leader) mbar_arrive_expect_tx(bar_l1_full, 2u * 4u * static_cast<uint32_t>(l1_rows) * 128u);
#pragma unroll
        for (int sl = 0; sl < 4; ++sl)
          tma2_load_2d(l1_base + sl * l1_pitch, &tmL1T, l1_full0, n0 + 64 * sl, static_cast<int>(rank) * l1_rows);
      }
      if (leader) {
        ok = __all_sync(0xffffffffu, bounded_wait<64>(bar_xh_full, k & 1u, env, kErrMmaWait) &&
                                         bounded_wait<64>(bar_l1_full, k & 1u, env, kErrMmaWait));
        if (!ok) break;
        tc_fence_after_sync();
        const bool first = tn == tn0, last = tn + 1 == tn1;
        if (first) {  // the buffer's previous row pair must have been read out
          const uint32_t uses = tb ? uses1 : uses0;
          ok = __all_sync(0xffffffffu, bounded_wait<64>(bar_t_empty + 8 * tb, (uses & 1u) ^ 1u, env, kErrMmaWait));
          if (!ok) break;
          tc_fence_after_sync();
        }
        if (issuer) {
          const uint32_t d = tmem_base + kMxTmemT + 64 * tb;
#pragma unroll
          for (int sl = 0; sl < 4; ++sl) {
#pragma unroll
            for (int kk = 0; kk < 4; ++kk)
              umma2_f16(d, umma_desc_k_sw128(xh_base + sl * kMxATile, 32 * kk), umma_desc_k_sw128(l1_base + sl * l1_pitch, 32 * kk),
                        idesc_t, (first && sl == 0 && kk == 0) ? 0u : 1u);
          }
          umma2_commit(bar_xh_empty);
          umma2_commit(peer_xh_empty);
          if (last) {
            umma2_commit(bar_t_full + 8 * tb);
            umma2_commit(peer_t_full + 8 * tb);
          }
        }
        if (last) {
          if (tb) ++uses1; else ++uses0;
          tb ^= 1u;
        }
      }
    }
  } else if (live && warp >= kMxEpiWarp0) {
    // ------------------------------------------------------------------ epilogue (both CTAs, own rows)
    const int ew = warp - kMxEpiWarp0;
    const int quarter = ew & 3, colblk = ew >> 2;
    const uint32_t acc_empty_leader = map_to_cta(bar_acc_empty, 0);
    Ring<1> ab;
    uint32_t kq = 0, tb = 0, t_uses0 = 0, t_uses1 = 0;   // FUSE: items done, T buffer, drains per buffer
    bool ok = true;
    for (int q = cluster_id; ok && q < num_runs; q += num_clusters)
    for (int tn = (q % runs_per_pair) * run, tn1 = min(tn + run, p.tiles_n); ok && tn < tn1; ++tn) {
      const int m0 = (2 * (q / runs_per_pair) + static_cast<int>(rank)) * kBM, n0 = tn * kMxBN;
      const int row = m0 + 32 * quarter + lane;
      // FUSE: the warp's 64 bias values and 64 reciprocal smoothing factors of the next layer go into a table of its
      // own in shared memory (the half of the L1' area that ranks up to 32 leave free) while the tile is still
      // being accumulated; from global memory each of them would be a long-latency load in front of its use.
      const bool use_tab = FUSE && nx.r2 <= 32;
      const uint32_t tab = l1_base + 8192 + static_cast<uint32_t>(ew) * 512;
      if (use_tab) {
        const int chq = n0 + 64 * colblk + 4 * (lane & 15);
        float4 t4 = make_float4(0.f, 0.f, 0.f, 0.f);
        if (chq < p.N) {
          if (lane >= 16) t4 = __ldg(reinterpret_cast<const float4*>(nx.rlam + chq));
          else if (p.bias) t4 = __ldg(reinterpret_cast<const float4*>(p.bias + chq));
        }
        __syncwarp();   // the previous item's reads of the table are done
        asm volatile("st.shared.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(tab + 16 * lane), "f"(t4.x), "f"(t4.y), "f"(t4.z), "f"(t4.w) : "memory");
        __syncwarp();
      }
      ok = bounded_wait(bar_acc_full, ab.parity, env, kErrEpilogueWait);
      if (!ok) break;
      tc_fence_after_sync();
      const uint32_t t_row = tmem_base + (static_cast<uint32_t>(32 * quarter) << 16) + 64 * colblk;
      uint32_t v[4][16];
#pragma unroll
      for (int c = 0; c < 4; ++c) tmem_ld_32x32b_x16(t_row + 16 * c, v[c]);
      tmem_wait_ld();
      tc_fence_before_sync();
      __syncwarp();
      if (lane == 0) mbar_arrive_remote(acc_empty_leader);
      const int ch0 = n0 + 64 * colblk;
      if (FUSE) {
        // The layer's output never reaches memory: bias, activation and BF16 rounding as the plain epilogue would
        // apply them, then the next layer's kernel 1 on the thread's 64 channels (two MX blocks).
        const bool with_t = nx.r2 > 0;
        if (with_t) {  // the previous item's T MMAs have read the x_hat tile
          ok = __all_sync(0xffffffffu, bounded_wait(bar_xh_empty, (kq & 1u) ^ 1u, env, kErrEpilogueWait));
          if (!ok) break;
        }
        const bool row_ok = row < p.M, ch_ok = ch0 < p.N;
        const int rr = 32 * quarter + lane;
        const uint32_t xrow = xh_base + colblk * kMxATile + (rr >> 3) * 1024 + (rr & 7) * 128;
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          const int ch = ch0 + 16 * c;
          uint32_t xw[8];
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            float4 b4 = make_float4(0.f, 0.f, 0.f, 0.f), l4 = b4;
            if (use_tab) {
              asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(b4.x), "=f"(b4.y), "=f"(b4.z), "=f"(b4.w) : "r"(tab + 64 * c + 16 * i));
              asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(l4.x), "=f"(l4.y), "=f"(l4.z), "=f"(l4.w) : "r"(tab + 256 + 64 * c + 16 * i));
            } else if (ch_ok) {
              if (p.bias) b4 = __ldg(reinterpret_cast<const float4*>(p.bias + ch) + i);
              l4 = __ldg(reinterpret_cast<const float4*>(nx.rlam + ch) + i);
            }
            const float bb[4] = {b4.x, b4.y, b4.z, b4.w}, ll[4] = {l4.x, l4.y, l4.z, l4.w};
            float xh[4];
#pragma unroll
            for (int e = 0; e < 4; e += 2) {
              float y0 = __uint_as_float(v[c][4 * i + e]) + bb[e], y1 = __uint_as_float(v[c][4 * i + e + 1]) + bb[e + 1];
              if (p.act != 0) {
                y0 = apply_activation(y0, p.act);
                y1 = apply_activation(y1, p.act);
              }
              const uint32_t yb = pack_bf16x2(y0, y1);                      // what the plain epilogue would store
              xh[e] = ch_ok ? __fmul_rn(__uint_as_float(yb << 16), ll[e]) : 0.0f;   // smoothing, as kernel 1 does it
              xh[e + 1] = ch_ok ? __fmul_rn(__uint_as_float(yb & 0xffff0000u), ll[e + 1]) : 0.0f;
              v[c][4 * i + e] = __float_as_uint(xh[e]);
              v[c][4 * i + e + 1] = __float_as_uint(xh[e + 1]);
            }
            xw[2 * i] = pack_bf16x2(xh[0], xh[1]);
            xw[2 * i + 1] = pack_bf16x2(xh[2], xh[3]);
          }
          if (with_t) {  // 128-byte swizzle of a K-major operand row: 16-byte chunk j sits at j ^ (row % 8)
            const uint32_t j0 = static_cast<uint32_t>(2 * c), sw = static_cast<uint32_t>(rr & 7);
            asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(xrow + ((j0 ^ sw) << 4)), "r"(xw[0]), "r"(xw[1]), "r"(xw[2]), "r"(xw[3]) : "memory");
            asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(xrow + (((j0 + 1) ^ sw) << 4)), "r"(xw[4]), "r"(xw[5]), "r"(xw[6]), "r"(xw[7]) : "memory");
          }
        }
        if (with_t) {
          fence_proxy_async_smem();   // generic-proxy stores -> visible to the tensor core's reads
          __syncwarp();
          if (lane == 0) mbar_arrive_remote_release(map_to_cta(bar_xh_full, 0));
        }
        if (row_ok && ch_ok) {
          const float rho2 = __ldg(nx.rho);
          uint4 w0, w1;
          const uint32_t ex0 = mxfp4_block32(v[0], v[1], rho2, w0);
          const uint32_t ex1 = mxfp4_block32(v[2], v[3], rho2, w1);
          uint4* cdst = reinterpret_cast<uint4*>(nx.codes + static_cast<size_t>(row) * (p.N >> 1) + (ch0 >> 1));
          cdst[0] = w0;
          cdst[1] = w1;
          const int sb = ch0 >> 5;   // even: the two exponent bytes are neighbours inside the atom
          uint8_t* sdst = nx.sfa + (static_cast<size_t>(row >> 7) * (p.N >> 7) + (sb >> 2)) * 512 + (row & 31) * 16 +
                          ((row & 127) >> 5) * 4 + (sb & 3);
          *reinterpret_cast<uint16_t*>(sdst) = static_cast<uint16_t>(ex0 | (ex1 << 8));
        }
        if (with_t) {
          const bool last = tn + 1 == tn1;
          if (last) {   // the run's T is complete after this item's MMAs: add it to the FP32 array
            const uint32_t uses = tb ? t_uses1 : t_uses0;
            ok = __all_sync(0xffffffffu, bounded_wait(bar_t_full + 8 * tb, uses & 1u, env, kErrEpilogueWait));
            if (!ok) break;
            tc_fence_after_sync();
            if (colblk == 0) {
              const uint32_t t_src = tmem_base + (static_cast<uint32_t>(32 * quarter) << 16) + kMxTmemT + 64 * tb;
              for (int cc = 0; cc < nx.r2 / 16; ++cc) {
                uint32_t tv[16];
                tmem_ld_32x32b_x16(t_src + 16 * cc, tv);
                tmem_wait_ld();
                if (row_ok) {
#pragma unroll
                  for (int j = 0; j < 16; ++j) atomicAdd(nx.t32 + static_cast<size_t>(row) * nx.r2 + 16 * cc + j, __uint_as_float(tv[j]));
                }
              }
              tc_fence_before_sync();
              __syncwarp();
              if (lane == 0) mbar_arrive_remote(map_to_cta(bar_t_empty + 8 * tb, 0));
            }
            if (tb) ++t_uses1; else ++t_uses0;
            tb ^= 1u;
          }
        }
        ++kq;
      } else if (p.yref != nullptr) {
        float e = 0.0f;
        if (row < p.M && ch0 < p.N) {
          const uint4* yr = reinterpret_cast<const uint4*>(p.yref + static_cast<size_t>(row) * p.N + ch0);
#pragma unroll
          for (int c = 0; c < 4; ++c) {
#pragma unroll
            for (int h = 0; h < 2; ++h) {
              const uint4 ref = __ldg(yr + 2 * c + h);
              const uint32_t rw[4] = {ref.x, ref.y, ref.z, ref.w};
#pragma unroll
              for (int i = 0; i < 8; ++i) {
                const int col = 8 * h + i;
                const float b = p.bias ? __ldg(p.bias + ch0 + 16 * c + col) : 0.0f;
                const float y_hat = __bfloat162float(__float2bfloat16_rn(apply_activation(__uint_as_float(v[c][col]) + b, p.act)));
                const float y_ref = __uint_as_float((i & 1) ? (rw[i >> 1] & 0xffff0000u) : (rw[i >> 1] << 16));
                const float d = y_ref - y_hat;
                e = fmaf(d, d, e);
              }
            }
          }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) e += __shfl_xor_sync(0xffffffffu, e, o);
        if (lane == 0) atomicAdd(p.sq_err, static_cast<double>(e));
      } else if (row < p.M && ch0 < p.N) {
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          const int ch = ch0 + 16 * c;
          uint4 o[2];
          uint32_t* ow = reinterpret_cast<uint32_t*>(o);
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            const float4 b4 = p.bias ? __ldg(reinterpret_cast<const float4*>(p.bias + ch) + i) : make_float4(0.f, 0.f, 0.f, 0.f);
            float y0 = __uint_as_float(v[c][4 * i]) + b4.x, y1 = __uint_as_float(v[c][4 * i + 1]) + b4.y;
            float y2 = __uint_as_float(v[c][4 * i + 2]) + b4.z, y3 = __uint_as_float(v[c][4 * i + 3]) + b4.w;
            if (p.act != 0) {
              y0 = apply_activation(y0, p.act);
              y1 = apply_activation(y1, p.act);
              y2 = apply_activation(y2, p.act);
              y3 = apply_activation(y3, p.act);
            }
            __nv_bfloat162 lo = __floats2bfloat162_rn(y0, y1);
            __nv_bfloat162 hi = __floats2bfloat162_rn(y2, y3);
            ow[2 * i] = *reinterpret_cast<uint32_t*>(&lo);
            ow[2 * i + 1] = *reinterpret_cast<uint32_t*>(&hi);
          }
          uint4* y = reinterpret_cast<uint4*>(p.Y + static_cast<size_t>(row) * p.N + ch);
          y[0] = o[0];
          y[1] = o[1];
        }
      }
      ab.advance();
    }
  }

  // ---------------------------------------------------------------------- common tail
  tc_fence_before_sync();
  __syncthreads();
  if (*s_abort) {
    const uint64_t t0 = global_timer_ns();
    while (global_timer_ns() - t0 < 200000ull) __nanosleep(1000);
    __syncthreads();
  }
  cluster_sync_all();  // nothing may still be in flight towards a CTA that is about to leave
  if (warp == 2) {
    tc_fence_after_sync();
    tmem_dealloc2(tmem_base, 512);
  }
}

// Weight pack kernels of the MXFP4 variant (run once per layer).
// L1 [K, r] BF16 -> L1 transposed [r, K]: the K-major B operand of the fused producer's T MMA.
__global__ void mx_transpose_l1_kernel(const uint16_t* __restrict__ l1, uint16_t* __restrict__ out, int K, int r) {
  const size_t idx = static_cast<size_t>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (idx >= static_cast<size_t>(K) * r) return;
  const int k = static_cast<int>(idx / r), c = static_cast<int>(idx % r);
  out[static_cast<size_t>(c) * K + k] = l1[idx];
}
// codes [K, N] (one E2M1 code per byte) -> [N, K/2], two codes per byte, even K in the low nibble.
__global__ void mx_pack_weight_kernel(const uint8_t* __restrict__ codes, uint8_t* __restrict__ out, int K, int N,
                                      int* __restrict__ bad) {
  const int n = blockIdx.x * blockDim.x + threadIdx.x;
  const int c = blockIdx.y;  // chunk of 32 consecutive K
  if (n >= N) return;
  uint32_t w[4] = {0, 0, 0, 0};
  bool oob = false;
  for (int o = 0; o < 32; ++o) {
    const uint32_t v = codes[static_cast<size_t>(32 * c + o) * N + n];
    oob |= v > 15u;
    w[o >> 3] |= (v & 15u) << (4 * (o & 7));
  }
  if (oob) atomicOr(bad, 1);
  *reinterpret_cast<uint4*>(out + static_cast<size_t>(n) * (K >> 1) + 16 * c) = make_uint4(w[0], w[1], w[2], w[3]);
}
// exps [K/32, N] (E8M0 bytes) -> scale atoms [N/128][K/128][512].
__global__ void mx_pack_wscale_kernel(const uint8_t* __restrict__ exps, uint8_t* __restrict__ out, int K, int N,
                                      int* __restrict__ bad) {
  const size_t idx = static_cast<size_t>(blockIdx.x) * blockDim.x + threadIdx.x;
  const int B = K / 32;
  if (idx >= static_cast<size_t>(B) * N) return;
  const int n = idx % N, b = idx / N;
  const uint8_t e = exps[idx];
  if (e == 0xFF) atomicOr(bad, 1);  // E8M0's NaN encoding
  out[(static_cast<size_t>(n >> 7) * (K / 128) + (b >> 2)) * 512 + (n & 31) * 16 + ((n & 127) >> 5) * 4 + (b & 3)] = e;
}
// Test-only decoders of the MXFP4 activation kernel's outputs.
__global__ void mx_decode_codes_kernel(const uint8_t* __restrict__ packed, uint8_t* __restrict__ codes, int M, int K) {
  const size_t idx = static_cast<size_t>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (idx >= static_cast<size_t>(M) * K) return;
  const uint8_t b = packed[idx >> 1];
  codes[idx] = (idx & 1) ? (b >> 4) : (b & 15);
}
__global__ void mx_decode_exps_kernel(const uint8_t* __restrict__ atoms, int atoms_k, uint8_t* __restrict__ exps, int M, int B) {
  const size_t idx = static_cast<size_t>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (idx >= static_cast<size_t>(M) * B) return;
  const int b = idx % B;
  const int m = idx / B;
  exps[idx] = atoms[(static_cast<size_t>(m >> 7) * atoms_k + (b >> 2)) * 512 + (m & 31) * 16 + ((m & 127) >> 5) * 4 + (b & 3)];
}

}  // namespace w4a4
