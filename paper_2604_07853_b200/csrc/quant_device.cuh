// Device helpers of the 1x128 / 128x128 block quantizers (Sec. 2.2), shared by the kernels that quantize.
#pragma once
#include "common.cuh"

namespace qarl {
namespace {

__device__ __forceinline__ uint32_t absmax_bf16x2(uint32_t m, uint32_t v) {
  return __vmaxu2(m, v & 0x7FFF7FFFu);  // per-halfword unsigned max of |x| bit patterns
}
__device__ __forceinline__ uint32_t absmax_u4(uint32_t m, const uint4& v) {
  m = absmax_bf16x2(m, v.x);
  m = absmax_bf16x2(m, v.y);
  m = absmax_bf16x2(m, v.z);
  return absmax_bf16x2(m, v.w);
}
__device__ __forceinline__ uint32_t fold_halves(uint32_t m) { return max(m & 0xFFFFu, m >> 16); }

// 8 bf16 (one uint4) -> 8 codes in two 32-bit words.
__device__ __forceinline__ void encode8(const uint4& v, float inv, uint32_t& c0, uint32_t& c1) {
  const float f0 = __fmul_rn(bf16_bits_to_f32(v.x & 0xFFFFu), inv), f1 = __fmul_rn(bf16_bits_to_f32(v.x >> 16), inv);
  const float f2 = __fmul_rn(bf16_bits_to_f32(v.y & 0xFFFFu), inv), f3 = __fmul_rn(bf16_bits_to_f32(v.y >> 16), inv);
  const float f4 = __fmul_rn(bf16_bits_to_f32(v.z & 0xFFFFu), inv), f5 = __fmul_rn(bf16_bits_to_f32(v.z >> 16), inv);
  const float f6 = __fmul_rn(bf16_bits_to_f32(v.w & 0xFFFFu), inv), f7 = __fmul_rn(bf16_bits_to_f32(v.w >> 16), inv);
  c0 = cvt_e4m3x4(f0, f1, f2, f3);
  c1 = cvt_e4m3x4(f4, f5, f6, f7);
}

}  // namespace
}  // namespace qarl
