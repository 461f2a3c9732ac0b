// Expansion of packed 4-bit weight codes to bf16 next to the tensor core (Dequant of Sec. 2.2),
// shared by the wide-tile and the decode-sized W4A16 GEMM kernels: both must produce the same bits.
#pragma once
#include <stdint.h>

namespace qarl {

// Two codes in bits [0,4) and [16,20) of `pair` -> bf16x2 of s * (q - z): 128 + q is exact in
// bf16 (0x4300 | q), the subtraction of 128 + z is exact, the product is rounded once.
__device__ __forceinline__ uint32_t dequant_pair(uint32_t pair, uint32_t zc2, uint32_t s2) {
  uint32_t t, d, v;
  asm("lop3.b32 %0, %1, 0x000F000F, 0x43004300, 0xEA;" : "=r"(t) : "r"(pair));  // (a & b) | c
  asm("sub.rn.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(t), "r"(zc2));
  asm("mul.rn.bf16x2 %0, %1, %2;" : "=r"(v) : "r"(d), "r"(s2));
  return v;
}

// Eight codes of one 32-bit word -> 16 bytes (eight bf16 in K order).
__device__ __forceinline__ uint4 dequant_word(uint32_t w, uint32_t zc2, uint32_t s2) {
  return make_uint4(dequant_pair(w, zc2, s2), dequant_pair(w >> 4, zc2, s2), dequant_pair(w >> 8, zc2, s2),
                    dequant_pair(w >> 12, zc2, s2));
}

// e2m1 codes (Sec. 2.2, floating-point quantization): sign | 2 exponent bits (bias 1) | 1 mantissa bit.
// Placed at bits 15 | 8..7 | 6 of a bf16, a code reads as its own value times 2^-126 (the code's
// subnormals 0 and 0.5 land on bf16 subnormals), so two exact-or-once-rounded multiplications give
// w^ = bf16(s * value): first by 2^a, exact, then by c = s 2^(126 - a); value has 2 significant bits and s
// 8, so the last product is the single rounding.  a is chosen per group so that both factors stay
// finite and normal for every bf16 s: a = min(127, E_s - 1) with E_s the exponent field of s.
__device__ __forceinline__ void fp4_group_consts(uint32_t s_bits, uint32_t& c1x2, uint32_t& c2x2) {
  const uint32_t es = (s_bits >> 7) & 0xFFu;
  const uint32_t a = min(127u, es - 1u);
  c1x2 = ((a + 127u) << 7) * 0x00010001u;
  c2x2 = ((s_bits & 0x7Fu) | ((es + 126u - a) << 7)) * 0x00010001u;
}
__device__ __forceinline__ uint32_t dequant_bits_fp4(uint32_t x6, uint32_t x12, uint32_t c1x2, uint32_t c2x2) {
  const uint32_t t = (x6 & 0x01C001C0u) | (x12 & 0x80008000u);
  uint32_t u, v;
  asm("mul.rn.bf16x2 %0, %1, %2;" : "=r"(u) : "r"(t), "r"(c1x2));
  asm("mul.rn.bf16x2 %0, %1, %2;" : "=r"(v) : "r"(u), "r"(c2x2));
  return v;
}
// Eight e2m1 codes of one 32-bit word (pairs in bits [4j, 4j+4) and [16+4j, 20+4j)) -> eight bf16 in K order.
__device__ __forceinline__ uint4 dequant_word_fp4(uint32_t w, uint32_t c1x2, uint32_t c2x2) {
  return make_uint4(dequant_bits_fp4(w << 6, w << 12, c1x2, c2x2), dequant_bits_fp4(w << 2, w << 8, c1x2, c2x2),
                    dequant_bits_fp4(w >> 2, w << 4, c1x2, c2x2), dequant_bits_fp4(w >> 6, w, c1x2, c2x2));
}

}  // namespace qarl
