// Kernel 1: fused smoothing + per-(token, 64-channel group) 4-bit quantization + code output
// + low-rank down-projection, one streaming pass over the BF16 activations (HBM bound).
//
//   Eq. 5      xh = f32(x) * (1/lambda)                      one FP32 multiply per element
//   Eq. 8      a  = max |xh| over the 64-channel group       quad shuffles
//   Eq. 9 / 4  s  = (rho * a) / 7 ,  is = 1 / s              IEEE divides, once per (row, group)
//   Eq. 3      q  = clip(rint(xh * is), -8, 7)               rounding by the 1.5*2^23 magic add (ties to even)
//   Eq. 7      T  = bf16(xh) L1                              mma.sync m16n8k16 BF16, FP32 accumulate
//
// Work split: a CTA of kQuantWarps warps owns 16 consecutive token rows per warp; all warps walk the K groups
// together, so the group's L1 fragments and smoothing factors are staged once per CTA.  Inside a warp,
// lane = 4*i + j owns rows i and i+8 and, within the group, channels
//      32*(j/2) + 8*(j%2) + [0,8)     and the same + 16,
// which is exactly the pair of 8-channel runs that fill two whole 32-bit words of the packed layout
// below, so no lane exchange is needed to pack.  The tensor-core K order is free (a dot product does
// not care about order), so the lane's 16 channels are used as-is as A-fragment slots and the L1
// fragments are laid out at pack time to match (see l1_fragment_channel()).
//
// K split (gridDim.y > 1): with few token rows there are too few 16-row warps to fill the machine, so the K groups
// are divided among gridDim.y CTAs per row block.  Codes and scales of different groups are independent; the
// partial sums of T go to an FP32 scratch [split][M][r] and t_reduce_kernel adds them in split order and writes
// the BF16 high | low pair.
//
// Code output, three formats (template parameter FORMAT):
//   kCodesE4M3    one E4M3 byte per code, row-major [M, K]: the tensor-core operand of kernel 2 as it is
//                 (fp8_codes.cuh), fetched by TMA straight into the swizzled operand tile;
//   kCodesPacked  nibble-packed INT4, half the bytes, for callers that want the compact form;
//   kCodesMxfp4   the MXFP4 variant of the layer (OCP MX v1.0: E2M1 elements, one E8M0 scale per 32 channels,
//                 shared exponent floor(log2(rho * block maximum)) - 2): two codes per byte, row-major
//                 [M, K/2], and the scale bytes in the 512-byte atoms the block-scaled tensor-core
//                 instruction wants in TMEM (see mx_gemm_kernel.cuh).
// Packed activation layout: per row, per 32 consecutive channels
// [32c, 32c+32) one 16-byte chunk of four 32-bit words; word w, byte b holds channel 32c + 4w + b in
// its LOW nibble and channel 32c + 16 + 4w + b in its HIGH nibble (two's complement nibbles).  With
// that interleave `word & 0x0F0F0F0F` and `(word >> 4) & 0x0F0F0F0F` are each four K-contiguous codes,
// one per byte.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "fp8_codes.cuh"

namespace w4a4 {

constexpr int kCodesPacked = 0, kCodesE4M3 = 1, kCodesMxfp4 = 2;
constexpr int kQuantRows = 16;      // token rows per CTA
// Warps per CTA (16 rows each).  Small CTAs spread evenly over the 148 SMs; the widest rank shares its
// larger L1 fragments among more warps.
constexpr int quantize_warps(int R) { return R >= 64 ? 4 : 2; }
constexpr int kStages = 3;          // depth of the cp.async rings (groups in flight = kStages - 1)

// Dynamic shared memory of quantize_kernel<R>: activation rings, smoothing-factor ring, L1 fragment ring.
constexpr size_t quantize_smem_bytes(int R) {
  return static_cast<size_t>(quantize_warps(R)) * kStages * 4 * 32 * 16 + kStages * 64 * 4 +
         static_cast<size_t>(kStages) * (4 * (R / 8) * 32 * 8);
}

// Channel (within its 64-group) that lane-in-quad j holds as its e-th element, e in [0,16).
__host__ __device__ constexpr int l1_fragment_channel(int j, int e) {
  return 32 * (j >> 1) + 8 * (j & 1) + (e < 8 ? e : e + 8);
}

__device__ __forceinline__ void mma_bf16_16816(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}

__device__ __forceinline__ uint4 ldg_stream_v4(const void* p) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
               : "l"(p));
  return v;
}

// Smooth 8 BF16 values (one 16-byte load) with 8 reciprocals.
__device__ __forceinline__ void smooth8(const uint4& raw, const float4& r0, const float4& r1, float* xh) {
  const float2 a = __fmul2_rn(make_float2(__uint_as_float(raw.x << 16), __uint_as_float(raw.x & 0xffff0000u)), make_float2(r0.x, r0.y));
  const float2 b = __fmul2_rn(make_float2(__uint_as_float(raw.y << 16), __uint_as_float(raw.y & 0xffff0000u)), make_float2(r0.z, r0.w));
  const float2 c = __fmul2_rn(make_float2(__uint_as_float(raw.z << 16), __uint_as_float(raw.z & 0xffff0000u)), make_float2(r1.x, r1.y));
  const float2 d = __fmul2_rn(make_float2(__uint_as_float(raw.w << 16), __uint_as_float(raw.w & 0xffff0000u)), make_float2(r1.z, r1.w));
  xh[0] = a.x; xh[1] = a.y; xh[2] = b.x; xh[3] = b.y; xh[4] = c.x; xh[5] = c.y; xh[6] = d.x; xh[7] = d.y;
}

// Group absolute maximum of the lane's 16 smoothed values, combined over the quad (= 64 channels).
__device__ __forceinline__ float quad_absmax16(const float* xh) {
  float a0 = fmaxf(fabsf(xh[0]), fabsf(xh[1])), a1 = fmaxf(fabsf(xh[2]), fabsf(xh[3]));
#pragma unroll
  for (int e = 4; e < 16; e += 2) {
    a0 = fmaxf(a0, fabsf(xh[e]));
    a1 = fmaxf(a1, fabsf(xh[e + 1]));
  }
  float a = fmaxf(a0, a1);
  a = fmaxf(a, __shfl_xor_sync(0xffffffffu, a, 1));
  a = fmaxf(a, __shfl_xor_sync(0xffffffffu, a, 2));
  return a;
}

// Eq. 8-9 / Eq. 4: s = (rho * a) / 7 and its reciprocal, both correctly rounded (IEEE); a == 0 -> 0, 0.
__device__ __forceinline__ void group_scale(float rho, float a, float& s, float& is) {
  s = 0.0f;
  is = 0.0f;
  if (a > 0.0f) {
    s = __fdiv_rn(__fmul_rn(rho, a), 7.0f);
    is = __frcp_rn(s);  // == 1.0f / s, round to nearest
  }
}

// Eq. 3 for the lane's 16 smoothed values of one row: code + 8 in [0, 15].
__device__ __forceinline__ void quantize16_offset(const float* xh, float is, uint32_t (&u)[16]) {
  // (float bits of z + 1.5*2^23 + 8) - bits(1.5*2^23), clamped.
#pragma unroll
  for (int e = 0; e < 16; ++e) {
    const float f = __fadd_rn(__fmul_rn(xh[e], is), 12582920.0f);
    u[e] = static_cast<uint32_t>(__viaddmin_s32_relu(__float_as_int(f), -0x4B400000, 15));
  }
}

// Quantize the lane's 16 values and return them as E4M3 bytes: .x/.y = elements 0..7 (channels coff .. +7),
// .z/.w = elements 8..15 (channels coff + 16 .. +23).
__device__ __forceinline__ uint4 quantize16_bytes(const float* xh, float is) {
  // Eq. 3: z = xh * is rounded to FP32, then to the nearest integer with ties to even (cvt.rni), then clamped to
  // [-8, 7]: cvt.pack.sat.s4 saturates two integers to 4 bits and shifts them in under the nibbles packed so far,
  // so the eight codes of a word take four instructions, element 0 in the lowest nibble.
  uint32_t n[2];
#pragma unroll
  for (int hh = 0; hh < 2; ++hh) {
    int v[8];
#pragma unroll
    for (int e = 0; e < 8; e += 2) {
      const float2 z = __fmul2_rn(make_float2(xh[8 * hh + e], xh[8 * hh + e + 1]), make_float2(is, is));
      v[e] = __float2int_rn(z.x);
      v[e + 1] = __float2int_rn(z.y);
    }
    uint32_t w;
    asm("cvt.pack.sat.s4.s32.b32 %0, %1, %2, %3;" : "=r"(w) : "r"(v[7]), "r"(v[6]), "r"(0));
    asm("cvt.pack.sat.s4.s32.b32 %0, %1, %2, %3;" : "=r"(w) : "r"(v[5]), "r"(v[4]), "r"(w));
    asm("cvt.pack.sat.s4.s32.b32 %0, %1, %2, %3;" : "=r"(w) : "r"(v[3]), "r"(v[2]), "r"(w));
    asm("cvt.pack.sat.s4.s32.b32 %0, %1, %2, %3;" : "=r"(w) : "r"(v[1]), "r"(v[0]), "r"(w));
    n[hh] = w ^ 0x88888888u;   // two's complement nibbles -> code + 8, the index the byte lookup takes
  }
  return make_uint4(e4m3_of_offset_nibbles4(n[0]), e4m3_of_offset_nibbles4(n[0] >> 16), e4m3_of_offset_nibbles4(n[1]),
                    e4m3_of_offset_nibbles4(n[1] >> 16));
}

// Quantize the lane's 16 smoothed values of one row (Eq. 3) and return its two packed words.
__device__ __forceinline__ uint2 quantize16(const float* xh, float is) {
  uint32_t u[16];
  quantize16_offset(xh, is, u);
  // One shift-add per code places its nibble: word w, byte b = low nibble u[4w+b], high nibble u[8+4w+b].
  uint32_t w0 = u[0], w1 = u[4];
#pragma unroll
  for (int b = 0; b < 4; ++b) {
    if (b > 0) {
      w0 += u[b] << (8 * b);
      w1 += u[4 + b] << (8 * b);
    }
    w0 += u[8 + b] << (8 * b + 4);
    w1 += u[12 + b] << (8 * b + 4);
  }
  return make_uint2(w0 ^ 0x88888888u, w1 ^ 0x88888888u);  // offset-binary -> two's complement nibbles
}

// Eight FP32 values -> eight E2M1 codes (round to nearest even, saturating at +-6), element 0 in the lowest nibble.
__device__ __forceinline__ uint32_t e2m1x8(const float* v) {
  uint32_t r;
  asm("{\n"
      ".reg .b8 t0, t1, t2, t3;\n"
      "cvt.rn.satfinite.e2m1x2.f32 t0, %2, %1;\n"
      "cvt.rn.satfinite.e2m1x2.f32 t1, %4, %3;\n"
      "cvt.rn.satfinite.e2m1x2.f32 t2, %6, %5;\n"
      "cvt.rn.satfinite.e2m1x2.f32 t3, %8, %7;\n"
      "mov.b32 %0, {t0, t1, t2, t3};\n"
      "}"
      : "=r"(r)
      : "f"(v[0]), "f"(v[1]), "f"(v[2]), "f"(v[3]), "f"(v[4]), "f"(v[5]), "f"(v[6]), "f"(v[7]));
  return r;
}

// MXFP4 conversion of the lane's 16 values of one row; they all lie in one 32-channel block, whose other half the
// neighbouring lane holds.  Returns the E8M0 exponent byte; packed codes in lo (elements 0..7) and hi (8..15).
__device__ __forceinline__ uint32_t mxfp4_block16(const float* xh, float rho, uint32_t& lo, uint32_t& hi) {
  float a0 = fmaxf(fabsf(xh[0]), fabsf(xh[1])), a1 = fmaxf(fabsf(xh[2]), fabsf(xh[3]));
#pragma unroll
  for (int e = 4; e < 16; e += 2) {
    a0 = fmaxf(a0, fabsf(xh[e]));
    a1 = fmaxf(a1, fabsf(xh[e + 1]));
  }
  float a = fmaxf(a0, a1);
  a = fmaxf(a, __shfl_xor_sync(0xffffffffu, a, 1));
  const uint32_t field = (__float_as_uint(__fmul_rn(rho, a)) >> 23) & 0xffu;   // exponent of the clip threshold (Eq. 8)
  const uint32_t ex = field > 2u ? field - 2u : 0u;                            // minus the exponent of E2M1's top binade
  const float inv = __uint_as_float((254u - ex) << 23);                        // 2^(127 - ex): exact scaling
  float v[16];
#pragma unroll
  for (int e = 0; e < 16; ++e) v[e] = __fmul_rn(xh[e], inv);
  lo = e2m1x8(v);
  hi = e2m1x8(v + 8);
  return ex;
}

// The token side of the GEMM's scale MMA for one (row, group): the scale as two BF16 pieces, s = h + m up to 2^-16
// relative, laid out [h, h, m, m] against the channel side's [w1, w2, w1, w2].
__device__ __forceinline__ uint2 sop_slots_activation(float s) {
  const __nv_bfloat16 h = __float2bfloat16_rn(s);
  const __nv_bfloat16 m = __float2bfloat16_rn(s - __bfloat162float(h));
  const uint32_t hb = __bfloat16_as_ushort(h), mb = __bfloat16_as_ushort(m);
  return make_uint2(hb | (hb << 16), mb | (mb << 16));
}

template <int R, int WARPS, int FORMAT>
// Sixteen resident warps per SM (at most 128 registers) at every rank, so that the 2048 warps of row blocks of the
// DiT shapes fit one wave: at 130-160 registers the wide ranks ran 1.15 waves.
__global__ void __launch_bounds__(32 * WARPS, 16 / WARPS)
quantize_kernel(const uint16_t* __restrict__ X, int M, int K, const float* __restrict__ rlam,
                const float* __restrict__ clip_table, int clip_index, const uint2* __restrict__ l1frag,
                uint8_t* __restrict__ codes, float* __restrict__ scales, int scales_ld,
                uint16_t* __restrict__ t_hilo, float* __restrict__ t_partial, uint2* __restrict__ a_sop) {
  constexpr int NT = R / 8;                          // n-tiles of the m16n8k16 MMA
  constexpr int kFragBytes = 4 * NT * 32 * 8;        // L1 fragments of one group (4 KiB at r = 32)
  constexpr int kFragChunks = kFragBytes / 16;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int qi = lane >> 2, qj = lane & 3;
  const int G = K >> 6;
  const int row0 = (blockIdx.x * WARPS + warp) * kQuantRows;
  const int rowA = row0 + qi, rowB = rowA + 8;
  const bool okA = rowA < M, okB = rowB < M;
  const float rho = __ldg(clip_table + clip_index);
  const int coff = 32 * (qj >> 1) + 8 * (qj & 1);  // lane's first channel inside a group

  const uint16_t* xa = X + static_cast<size_t>(okA ? rowA : 0) * K + coff;
  const uint16_t* xb = X + static_cast<size_t>(okB ? rowB : 0) * K + coff;

  float acc[NT > 0 ? NT : 1][4];
#pragma unroll
  for (int nt = 0; nt < (NT > 0 ? NT : 1); ++nt) acc[nt][0] = acc[nt][1] = acc[nt][2] = acc[nt][3] = 0.0f;

  // Everything a group needs is streamed through shared-memory rings with cp.async, kStages - 1 groups
  // ahead of the one being processed:
  //   xring   per warp: the 16 rows x 64 channels of activations (2 KiB); every lane reads back only the
  //           4 x 16 bytes it requested itself ([piece][lane] layout, conflict free, no barrier needed);
  //   fring   per CTA: the group's L1 fragments, shared by the CTA's warps (they all walk the same groups,
  //           each on its own 16 rows), so L1 crosses L2 once per 64 rows instead of once per 16;
  //   lring   per CTA: the group's 64 reciprocal smoothing factors.
  extern __shared__ __align__(16) uint8_t quant_smem[];
  typedef uint4 (*XRing)[kStages][4][32];
  typedef uint4 (*FRing)[kFragChunks > 0 ? kFragChunks : 1];
  typedef float (*LRing)[64];
  XRing xring = reinterpret_cast<XRing>(quant_smem);
  LRing lring = reinterpret_cast<LRing>(quant_smem + WARPS * kStages * 4 * 32 * 16);
  FRing fring = reinterpret_cast<FRing>(quant_smem + WARPS * kStages * 4 * 32 * 16 + kStages * 64 * 4);
  const uint32_t xring0 = static_cast<uint32_t>(__cvta_generic_to_shared(&xring[warp][0][0][lane]));
  auto issue = [&](int gg, int stage) {
    const uint32_t dst = xring0 + stage * (4 * 32 * 16);
    const uint32_t szA = okA ? 16u : 0u, szB = okB ? 16u : 0u;  // rows past M are zero-filled
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(xa + 64 * gg), "r"(szA) : "memory");
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst + 512), "l"(xa + 64 * gg + 16), "r"(szA) : "memory");
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst + 1024), "l"(xb + 64 * gg), "r"(szB) : "memory");
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst + 1536), "l"(xb + 64 * gg + 16), "r"(szB) : "memory");
    if constexpr (NT > 0) {
      const uint4* src = reinterpret_cast<const uint4*>(l1frag) + static_cast<size_t>(gg) * kFragChunks;
      for (int c = threadIdx.x; c < kFragChunks; c += (32 * WARPS)) {
        const uint32_t d = static_cast<uint32_t>(__cvta_generic_to_shared(&fring[stage][c]));
        asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(d), "l"(src + c) : "memory");
      }
    }
    if (threadIdx.x < 16) {
      const uint32_t d = static_cast<uint32_t>(__cvta_generic_to_shared(&lring[stage][4 * threadIdx.x]));
      asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(d), "l"(rlam + 64 * gg + 4 * threadIdx.x) : "memory");
    }
  };
  // This CTA's share of the groups (all of them unless the launch splits K).
  const int g_per_split = (G + gridDim.y - 1) / gridDim.y;
  const int g_begin = blockIdx.y * g_per_split;
  const int g_end = min(G, g_begin + g_per_split);
#pragma unroll
  for (int d = 0; d < kStages - 1; ++d) {
    if (g_begin + d < g_end) issue(g_begin + d, d);
    asm volatile("cp.async.commit_group;" ::: "memory");
  }
  int stage = 0;
  for (int g = g_begin; g < g_end; ++g) {
    // This thread's copies for group g have landed; after the barrier so have everyone's, and every warp
    // has finished group g - 1, whose ring slot the prefetch below overwrites.
    asm volatile("cp.async.wait_group %0;" ::"n"(kStages - 2) : "memory");
    __syncthreads();
    {
      int pstage = stage + kStages - 1;
      if (pstage >= kStages) pstage -= kStages;
      if (g + kStages - 1 < g_end) issue(g + kStages - 1, pstage);
      asm volatile("cp.async.commit_group;" ::: "memory");
    }
    const uint4* slot = &xring[warp][stage][0][lane];
    const uint4 ca0 = slot[0], ca1 = slot[32], cb0 = slot[64], cb1 = slot[96];
    const float4* rl = reinterpret_cast<const float4*>(&lring[stage][coff]);
    const float4 l0 = rl[0], l1 = rl[1], l4 = rl[4], l5 = rl[5];
    float xhA[16], xhB[16];
    smooth8(ca0, l0, l1, xhA);
    smooth8(ca1, l4, l5, xhA + 8);
    smooth8(cb0, l0, l1, xhB);
    smooth8(cb1, l4, l5, xhB + 8);

    if constexpr (FORMAT == kCodesMxfp4) {
      // `scales` is the scale-byte workspace here: per 128-row block and per 4 scale blocks (128 channels) one
      // 512-byte atom, byte (row % 32) * 16 + (row % 128 / 32) * 4 + (scale block % 4); scales_ld = atoms per row block.
      uint32_t loA, hiA, loB, hiB;
      const uint32_t exA = mxfp4_block16(xhA, rho, loA, hiA), exB = mxfp4_block16(xhB, rho, loB, hiB);
      uint8_t* ca = codes + static_cast<size_t>(rowA) * (K >> 1) + 32 * g + (coff >> 1);
      uint8_t* cb = codes + static_cast<size_t>(rowB) * (K >> 1) + 32 * g + (coff >> 1);
      if (okA) {
        *reinterpret_cast<uint32_t*>(ca) = loA;
        *reinterpret_cast<uint32_t*>(ca + 8) = hiA;
      }
      if (okB) {
        *reinterpret_cast<uint32_t*>(cb) = loB;
        *reinterpret_cast<uint32_t*>(cb + 8) = hiB;
      }
      if ((qj & 1) == 0) {
        uint8_t* sf = reinterpret_cast<uint8_t*>(scales);
        const int sb = 2 * g + (qj >> 1);  // scale block of this lane's channels
        const size_t atom_col = static_cast<size_t>(sb >> 2) * 512 + (sb & 3);
        if (okA) sf[(static_cast<size_t>(rowA >> 7) * scales_ld) * 512 + atom_col + (rowA & 31) * 16 + ((rowA & 127) >> 5) * 4] = static_cast<uint8_t>(exA);
        if (okB) sf[(static_cast<size_t>(rowB >> 7) * scales_ld) * 512 + atom_col + (rowB & 31) * 16 + ((rowB & 127) >> 5) * 4] = static_cast<uint8_t>(exB);
      }
    } else {
    // Even lanes of the quad derive row A's scale, odd lanes row B's; one shuffle shares the reciprocals.
    const float aA = quad_absmax16(xhA), aB = quad_absmax16(xhB);
    float s_mine, is_mine;
    group_scale(rho, (qj & 1) ? aB : aA, s_mine, is_mine);
    const float is_other = __shfl_xor_sync(0xffffffffu, is_mine, 1);
    const float isA = (qj & 1) ? is_other : is_mine, isB = (qj & 1) ? is_mine : is_other;
    if constexpr (FORMAT == kCodesE4M3) {
      const uint4 bA = quantize16_bytes(xhA, isA);
      const uint4 bB = quantize16_bytes(xhB, isB);
      uint8_t* ca = codes + static_cast<size_t>(rowA) * K + 64 * g + coff;
      uint8_t* cb = codes + static_cast<size_t>(rowB) * K + 64 * g + coff;
      if (okA) {
        *reinterpret_cast<uint2*>(ca) = make_uint2(bA.x, bA.y);
        *reinterpret_cast<uint2*>(ca + 16) = make_uint2(bA.z, bA.w);
      }
      if (okB) {
        *reinterpret_cast<uint2*>(cb) = make_uint2(bB.x, bB.y);
        *reinterpret_cast<uint2*>(cb + 16) = make_uint2(bB.z, bB.w);
      }
    } else {
      const uint2 wA = quantize16(xhA, isA);
      const uint2 wB = quantize16(xhB, isB);
      const size_t cpitch = static_cast<size_t>(K >> 1);
      if (okA) *reinterpret_cast<uint2*>(codes + rowA * cpitch + 32 * g + 8 * qj) = wA;
      if (okB) *reinterpret_cast<uint2*>(codes + rowB * cpitch + 32 * g + 8 * qj) = wB;
    }
    // Scales are stored group-major ([G][scales_ld]): kernel 2 fetches a (2 groups x 128 rows) block by TMA.
    if (qj == 0 && okA) scales[static_cast<size_t>(g) * scales_ld + rowA] = s_mine;
    if (qj == 1 && okB) scales[static_cast<size_t>(g) * scales_ld + rowB] = s_mine;
    if (a_sop != nullptr && ((qj == 0 && okA) || (qj == 1 && okB))) {
      // The scale once more, as four BF16 slots of the operand from which the GEMM's tensor core forms sx * sw:
      // 2 KiB shared-memory images per (128 rows, 2 groups), [8-row group][8 rows][group parity][8 bytes].
      const int row = qj == 0 ? rowA : rowB;
      const size_t image = static_cast<size_t>(row >> 7) * ((G + 1) >> 1) + (g >> 1);
      a_sop[image * 256 + ((row & 127) >> 3) * 16 + (row & 7) * 2 + (g & 1)] = sop_slots_activation(s_mine);
    }
    }

    if constexpr (NT > 0) {
      // Fragment storage: [i][n-tile pair][lane] as uint4 = (b0, b1) of n-tile 2p, (b0, b1) of n-tile 2p + 1.
      const uint4* lf = &fring[stage][lane];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        uint32_t a[4];
        a[0] = pack_bf16x2(xhA[4 * i], xhA[4 * i + 1]);
        a[1] = pack_bf16x2(xhB[4 * i], xhB[4 * i + 1]);
        a[2] = pack_bf16x2(xhA[4 * i + 2], xhA[4 * i + 3]);
        a[3] = pack_bf16x2(xhB[4 * i + 2], xhB[4 * i + 3]);
#pragma unroll
        for (int np = 0; np < NT / 2; ++np) {
          const uint4 b = lf[(i * (NT / 2) + np) * 32];
          mma_bf16_16816(acc[2 * np], a, b.x, b.y);
          mma_bf16_16816(acc[2 * np + 1], a, b.z, b.w);
        }
      }
    }
    if (++stage == kStages) stage = 0;
  }

  if constexpr (NT > 0) {
    // Each warp owns its 16 rows over all of K (or over its split of K): T, or its partial sum, is complete in
    // the accumulators.  Unsplit: store it as a BF16 high part and the BF16 rounding of the remainder
    // ([T_hi | T_lo], two values per 32-bit store).  Split: store the FP32 partial sums for t_reduce_kernel.
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
      const int c = 8 * nt + 2 * qj;
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        const int row = h ? rowB : rowA;
        if (row < M) {
          const float t0 = acc[nt][2 * h], t1 = acc[nt][2 * h + 1];
          if (gridDim.y > 1) {
            *reinterpret_cast<float2*>(t_partial + (static_cast<size_t>(blockIdx.y) * M + row) * R + c) = make_float2(t0, t1);
            continue;
          }
          const __nv_bfloat16 h0 = __float2bfloat16_rn(t0), h1 = __float2bfloat16_rn(t1);
          const uint32_t hi = pack_bf16x2(__bfloat162float(h0), __bfloat162float(h1));
          const uint32_t lo = pack_bf16x2(t0 - __bfloat162float(h0), t1 - __bfloat162float(h1));
          uint16_t* dst = t_hilo + static_cast<size_t>(row) * (2 * R);
          *reinterpret_cast<uint32_t*>(dst + c) = hi;
          *reinterpret_cast<uint32_t*>(dst + R + c) = lo;
        }
      }
    }
  }
}

// Sum of the K splits' partial T (in split order), written as the BF16 high | low pair kernel 2 reads.
static __global__ void t_reduce_kernel(const float* __restrict__ t_partial, int splits, int M, int r, uint16_t* __restrict__ t_hilo) {
  const size_t idx = static_cast<size_t>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (idx >= static_cast<size_t>(M) * r) return;
  float t = 0.0f;
  for (int s = 0; s < splits; ++s) t += t_partial[static_cast<size_t>(s) * M * r + idx];
  const size_t row = idx / r;
  const int c = static_cast<int>(idx % r);
  const __nv_bfloat16 hi = __float2bfloat16_rn(t);
  const __nv_bfloat16 lo = __float2bfloat16_rn(t - __bfloat162float(hi));
  t_hilo[row * 2 * r + c] = *reinterpret_cast<const uint16_t*>(&hi);
  t_hilo[row * 2 * r + r + c] = *reinterpret_cast<const uint16_t*>(&lo);
}

// Number of K splits for a launch of `row_ctas` row blocks over G groups on a device with `sms` SMs: enough CTAs
// for about three per SM, at most kMaxKSplits, and only while the partial sums of T fit the scratch
// (M <= kKSplitMaxRows).
constexpr int kMaxKSplits = 8;
constexpr int kKSplitMaxRows = 8192;
inline int quantize_k_splits(int row_ctas, int G, int M, int sms) {
  if (M > kKSplitMaxRows || row_ctas >= 2 * sms) return 1;
  int s = (3 * sms + row_ctas - 1) / row_ctas;
  if (s > kMaxKSplits) s = kMaxKSplits;
  if (s > G) s = G;
  return s < 1 ? 1 : s;
}

}  // namespace w4a4
