// 4-bit codes as FP8 (E4M3) tensor-core operands.
//
// sm_100a has no 4-bit integer MMA, and its 8-bit integer MMA (kind::i8) leaves int32 partial sums that the
// epilogue must convert to FP32 one by one.  The codes of Eq. 3 are the integers -8 .. 7, all of which E4M3
// represents exactly, and the products and 64-term sums of such integers (|sum| <= 4096) are exact in the
// FP32 accumulators of tcgen05.mma kind::f8f6f4.  Feeding the codes as E4M3 bytes therefore yields the same
// per-group partial sums P of Eq. 7, already in FP32.
//
// Both kernels translate "code + 8" (a nibble u in [0, 15]) to its E4M3 byte with the same byte-permute
// lookup: two 8-entry tables held in two registers each, selected by the low three bits of every nibble,
// and a byte mask derived from the nibble's top bit that picks between them.
#pragma once

#include <stdint.h>

namespace w4a4 {

// E4M3 (1 sign, 4 exponent bits with bias 7, 3 mantissa bits) of c = u - 8, entry u in byte (u % 4) of word u / 4.
//   c:    -8    -7    -6    -5    -4    -3    -2    -1     0     1     2     3     4     5     6     7
//   byte: 0xD0  0xCE  0xCC  0xCA  0xC8  0xC4  0xC0  0xB8   0x00  0x38  0x40  0x44  0x48  0x4A  0x4C  0x4E
constexpr uint32_t kE4m3Neg0 = 0xCACCCED0u, kE4m3Neg1 = 0xB8C0C4C8u;   // u = 0..3, 4..7
constexpr uint32_t kE4m3Pos0 = 0x44403800u, kE4m3Pos1 = 0x4E4C4A48u;   // u = 8..11, 12..15

__device__ __forceinline__ uint32_t prmt(uint32_t a, uint32_t b, uint32_t sel) {
  uint32_t d;
  asm("prmt.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(sel));
  return d;
}

// Four nibbles u0..u3 in bits [0,16) of `s` (higher bits are ignored) -> the four E4M3 bytes of u_i - 8,
// u0 in the lowest byte.
__device__ __forceinline__ uint32_t e4m3_of_offset_nibbles4(uint32_t s) {
  const uint32_t idx = s & 0x7777u;
  const uint32_t neg = prmt(kE4m3Neg0, kE4m3Neg1, idx);
  const uint32_t pos = prmt(kE4m3Pos0, kE4m3Pos1, idx);
  const uint32_t is_pos = prmt(0x0000FF00u, 0u, (s >> 3) & 0x1111u);   // 0xFF where the nibble is >= 8
  return (pos & is_pos) | (neg & ~is_pos);
}

// Inverse, for the test-only decoders: the integer value of an E4M3 byte that encodes one.
__host__ __device__ inline int e4m3_integer_value(uint8_t b) {
  const int e = (b >> 3) & 15, f = b & 7;
  const float mag = e == 0 ? static_cast<float>(f) * 0.001953125f /* 2^-9 */
                           : (1.0f + static_cast<float>(f) * 0.125f) * static_cast<float>(1u << e) * 0.0078125f /* 2^-7 */;
  const int v = static_cast<int>(mag);
  return (b & 0x80) ? -v : v;
}

}  // namespace w4a4
