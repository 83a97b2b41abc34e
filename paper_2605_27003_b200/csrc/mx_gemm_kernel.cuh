// Kernel 2 of the MXFP4 variant: block-scaled FP4 GEMM + low-rank up-projection + bias + BF16 store.
//
//   Y[m,n] = sum_b 2^(ea[m,b]-127) 2^(ew[b,n]-127) sum_{k in block b} a[m,k] w[k,n]  +  sum_j T[m,j] L2[j,n]  +  b[n]
//
// a, w are E2M1 elements, ea / ew the E8M0 exponents of their 32-element blocks along K (OCP MX v1.0, the data
// format the paper's Table 1 names).  tcgen05.mma kind::mxf4.block_scale applies both block scales inside the
// tensor core and accumulates in FP32, so -- unlike the INT4 kernel -- nothing is rescaled on the CUDA cores and
// the whole K extent accumulates into one TMEM tile; the epilogue runs once per output tile.
//
// Persistent kernel, one CTA per SM, 128 x 256 output tiles, column tile fastest.  At the FP4 rate the tensor
// core consumes operands faster than L2 and the shared-memory port deliver them, so the tile is as wide as TMEM
// allows (operand bytes per MAC fall by a quarter against 128 x 128).  Warp roles:
//   warp 0      producer (one lane): per stage of 256 K elements one TMA each for the packed A tile (128 rows x
//               128 bytes) and B tile (256 rows x 128 bytes), 128-byte swizzle, and bulk copies for their scale
//               bytes (1 KiB per 128 rows: two 512-byte atoms, the layout the tensor core wants); the BF16
//               low-rank operands T and L2 go through the same ring first.
//   warp 1      MMA issuer (one lane): per stage six tcgen05.cp (scale atoms, shared memory -> TMEM: 32 lanes x
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
// Every wait is bounded exactly as in gemm_kernel.cuh (whose Ring / bounded_wait helpers are used here).
#pragma once

#include <cuda_bf16.h>
#include <stdint.h>

#include "gemm_kernel.cuh"
#include "ptx.cuh"

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
};

// One lane of a converged warp.  The MMA warp runs its loop with all lanes (waits included) and only predicates
// the tcgen05 instructions on this: everything they take as operands then stays warp-uniform for the compiler,
// which keeps descriptors and addresses in uniform registers instead of converting them per instruction
// (elect_one_lane() comes from gemm_kernel.cuh).

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
  const WaitEnv env{p.err, s_abort};

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
__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ uint32_t map_to_cta(uint32_t smem_addr, uint32_t cta_rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(smem_addr), "r"(cta_rank));
  return r;
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// Relaxed on purpose: the arrive only hands TMEM columns back (tcgen05.wait::ld has completed the reads, the
// tcgen05 fence orders them); a release at cluster scope would also wait for the warp's earlier global stores
// (the previous tile's outputs) to become visible, which cost about 1200 clocks per tile.
__device__ __forceinline__ void mbar_arrive_remote(uint32_t cluster_addr) {
  asm volatile("mbarrier.arrive.relaxed.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
// 2D tiled load into this CTA's shared memory whose byte count is reported to `bar_cluster_addr`, a barrier of
// this CTA or of the other CTA of the pair.
__device__ __forceinline__ void tma2_load_2d(uint32_t dst_smem, const CUtensorMap* tm, uint32_t bar_cluster_addr, int c0, int c1) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(dst_smem), "l"(reinterpret_cast<uint64_t>(tm)), "r"(bar_cluster_addr), "r"(c0), "r"(c1)
      : "memory");
}
__device__ __forceinline__ void tmem_alloc2(uint32_t smem_result, uint32_t ncols) {
  asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_result), "r"(ncols) : "memory");
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc2(uint32_t taddr, uint32_t ncols) {
  asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
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
__device__ __forceinline__ void umma2_f16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n"
      ".reg .pred p;\n"
      "setp.ne.b32 p, %4, 0;\n"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n"
      "}\n" ::"r"(d_tmem),
      "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// Arrives on the mbarrier at `cluster_addr` (this CTA's or the neighbour's) once the pair's MMAs issued so far are done.
__device__ __forceinline__ void umma2_commit(uint32_t cluster_addr) {
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(cluster_addr) : "memory");
}

constexpr int kMx2Stages = 6;
constexpr uint32_t kMx2BHalf = kMxBTile / 2;                                  // 16 KiB: this CTA's 128 rows of B
constexpr uint32_t kMx2StageBytes = kMxATile + kMx2BHalf + 3 * kMxSfTile;      // 35 KiB
constexpr uint32_t kMx2NumBarriers = 2 * kMx2Stages + 2;
constexpr uint32_t kMx2SmemBytes = 1024 + kMx2Stages * kMx2StageBytes + kMx2NumBarriers * 8 + 16;
static_assert(kMx2StageBytes % 1024 == 0, "operand tiles must stay 1024-byte aligned");

__global__ void __launch_bounds__(kMxThreads, 1)
mx_gemm2_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmBhalf,
                const __grid_constant__ CUtensorMap tmT, const __grid_constant__ CUtensorMap tmL2half,
                const __grid_constant__ CUtensorMap tmSFA, const __grid_constant__ CUtensorMap tmSFB, const MxGemmParams p) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* smem = smem_raw + (smem_base - smem_u32(smem_raw));
  const uint32_t bar_base = smem_base + kMx2Stages * kMx2StageBytes;
  const uint32_t bar_full = bar_base;
  const uint32_t bar_empty = bar_full + 8 * kMx2Stages;
  const uint32_t bar_acc_full = bar_empty + 8 * kMx2Stages;
  const uint32_t bar_acc_empty = bar_acc_full + 8;
  const uint32_t misc_off = (bar_acc_empty + 8) - smem_base;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + misc_off);
  volatile int* s_abort = reinterpret_cast<volatile int*>(smem + misc_off + 4);

  const int warp = __shfl_sync(0xffffffffu, static_cast<int>(threadIdx.x >> 5), 0), lane = threadIdx.x & 31;  // provably warp-uniform
  const uint32_t rank = cluster_ctarank();
  const bool leader = rank == 0;
  const int n_k_stages = p.K / kMxBK;
  const int n_lr_stages = p.r > 0 ? (2 * p.r + 63) / 64 : 0;
  const int num_items = ((p.tiles_m + 1) / 2) * p.tiles_n;
  const int cluster_id = blockIdx.x >> 1, num_clusters = gridDim.x >> 1;
  const WaitEnv env{p.err, s_abort};

  if (threadIdx.x == 0) {
    *s_abort = (*reinterpret_cast<volatile int*>(p.err) != 0) ? 1 : 0;
    for (int i = 0; i < kMx2Stages; ++i) {
      mbar_init(bar_full + 8 * i, 1);
      mbar_init(bar_empty + 8 * i, 1);
    }
    mbar_init(bar_acc_full, 1);
    mbar_init(bar_acc_empty, 2 * kMxEpiWarps);
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
    Ring<kMx2Stages> rg;
    bool ok = true;
    for (int item = cluster_id; ok && item < num_items; item += num_clusters) {
      const int tm = 2 * (item / p.tiles_n) + static_cast<int>(rank), tn = item % p.tiles_n;
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
    Ring<kMx2Stages> rg;
    Ring<1> ab;
    bool ok = true;
    for (int item = cluster_id; ok && item < num_items; item += num_clusters) {
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
  } else if (live && warp >= kMxEpiWarp0) {
    // ------------------------------------------------------------------ epilogue (both CTAs, own rows)
    const int ew = warp - kMxEpiWarp0;
    const int quarter = ew & 3, colblk = ew >> 2;
    const uint32_t acc_empty_leader = map_to_cta(bar_acc_empty, 0);
    Ring<1> ab;
    bool ok = true;
    for (int item = cluster_id; ok && item < num_items; item += num_clusters) {
      const int m0 = (2 * (item / p.tiles_n) + static_cast<int>(rank)) * kBM, n0 = (item % p.tiles_n) * kMxBN;
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
      if (lane == 0) mbar_arrive_remote(acc_empty_leader);
      const int ch0 = n0 + 64 * colblk;
      if (p.yref != nullptr) {
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
