// Block quantizers (Sec. 2.2, floating-point quantization): per block amax -> s = amax/448 ->
// e4m3 codes, for 128x128 weight blocks and 1x128 activation groups.  Both kernels are
// HBM-bound: 128-bit loads, 128-bit stores, every input byte read once.
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

// One CTA per 128x128 block.  256 threads; a thread owns 16 contiguous elements of a row
// (8 threads per row, 32 rows per pass, 4 passes), kept in registers between the amax
// reduction and the encode so the block is read from HBM once.
__global__ void __launch_bounds__(256) quantize_weight_kernel(const uint16_t* __restrict__ w, int64_t N, int64_t K,
                                                              uint8_t* __restrict__ codes,
                                                              float* __restrict__ scales) {
  pdl_trigger();
  pdl_wait();
  const int64_t kb = K / kBlock, nb = N / kBlock;
  const int64_t blk = blockIdx.x;
  const int64_t bk = blk % kb, bn = (blk / kb) % nb, e = blk / (kb * nb);
  const int tid = threadIdx.x;
  const int r0 = tid >> 3, c16 = (tid & 7) * 16;
  const int64_t base = (e * N + bn * kBlock) * K + bk * kBlock + c16;

  uint4 v[4][2];
  uint32_t m = 0;
#pragma unroll
  for (int p = 0; p < 4; ++p) {
    const uint4* src = reinterpret_cast<const uint4*>(w + base + static_cast<int64_t>(r0 + 32 * p) * K);
    v[p][0] = __ldg(src);
    v[p][1] = __ldg(src + 1);
  }
#pragma unroll
  for (int p = 0; p < 4; ++p) {
    m = absmax_u4(m, v[p][0]);
    m = absmax_u4(m, v[p][1]);
  }
  m = fold_halves(m);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) m = max(m, __shfl_xor_sync(0xFFFFFFFFu, m, o));
  __shared__ uint32_t warp_max[8];
  if ((tid & 31) == 0) warp_max[tid >> 5] = m;
  __syncthreads();
  m = warp_max[0];
#pragma unroll
  for (int i = 1; i < 8; ++i) m = max(m, warp_max[i]);

  float inv;
  const float s = block_scale(bf16_bits_to_f32(m), &inv);
  if (tid == 0) scales[blk] = s;
#pragma unroll
  for (int p = 0; p < 4; ++p) {
    uint4 out;
    encode8(v[p][0], inv, out.x, out.y);
    encode8(v[p][1], inv, out.z, out.w);
    *reinterpret_cast<uint4*>(codes + base + static_cast<int64_t>(r0 + 32 * p) * K) = out;
  }
}

// 8 threads per 1x128 group (16 elements each).  With dst_rows the codes and scale of input
// row t are written to `fanout` output rows (the token's positions in expert-sorted order).
__global__ void __launch_bounds__(256) quantize_act_kernel(const uint16_t* __restrict__ x, int64_t M, int64_t K,
                                                           int64_t ldx, uint8_t* __restrict__ codes,
                                                           float* __restrict__ scales,
                                                           const int32_t* __restrict__ dst_rows, int fanout,
                                                           int64_t dst_rows_total,
                                                           const float* __restrict__ pair_w,
                                                           float* __restrict__ sorted_w) {
  pdl_trigger();
  pdl_wait();
  const int64_t kb = K / kBlock;
  const int64_t gid = (static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x) >> 3;
  const bool live = gid < M * kb;
  const int64_t g = live ? gid : 0;
  const int64_t row = g / kb, b = g % kb;
  const int sub = threadIdx.x & 7;
  const uint4* src = reinterpret_cast<const uint4*>(x + row * ldx + b * kBlock + sub * 16);
  uint4 v0 = make_uint4(0, 0, 0, 0), v1 = v0;
  if (live) {
    v0 = __ldg(src);
    v1 = __ldg(src + 1);
  }
  uint32_t m = fold_halves(absmax_u4(absmax_u4(0, v0), v1));
#pragma unroll
  for (int o = 4; o > 0; o >>= 1) m = max(m, __shfl_xor_sync(0xFFFFFFFFu, m, o));
  float inv;
  const float s = block_scale(bf16_bits_to_f32(m), &inv);
  uint4 out;
  encode8(v0, inv, out.x, out.y);
  encode8(v1, inv, out.z, out.w);
  if (!live) return;
  if (dst_rows == nullptr) {
    *reinterpret_cast<uint4*>(codes + row * K + b * kBlock + sub * 16) = out;
    if (sub == 0) scales[row * kb + b] = s;
  } else {
    for (int j = 0; j < fanout; ++j) {
      // clamped: a pair with a bad expert id has no sorted position and leaves this entry stale
      const int64_t d = min(max(static_cast<int64_t>(dst_rows[row * fanout + j]), int64_t(0)), dst_rows_total - 1);
      *reinterpret_cast<uint4*>(codes + d * K + b * kBlock + sub * 16) = out;
      if (sub == 0) scales[d * kb + b] = s;
      if (sub == 0 && b == 0 && sorted_w != nullptr) sorted_w[d] = pair_w[row * fanout + j];
    }
  }
}

}  // namespace

cudaError_t launch_quantize_weight(const Launch& L, const uint16_t* w, int64_t E, int64_t N, int64_t K,
                                   uint8_t* codes, float* scales) {
  const int64_t blocks = E * (N / kBlock) * (K / kBlock);
  if (blocks == 0) return cudaSuccess;
  ++*L.launches;
  return launch_pdl(quantize_weight_kernel, static_cast<unsigned>(blocks), 256, 0, L.stream, w, N, K, codes, scales);
}

cudaError_t launch_quantize_act(const Launch& L, const uint16_t* x, int64_t M, int64_t K, int64_t ldx,
                                uint8_t* codes, float* scales, const int32_t* dst_rows, int fanout,
                                const float* pair_w, float* sorted_w) {
  const int64_t groups = M * (K / kBlock);
  if (groups == 0) return cudaSuccess;
  const int64_t blocks = (groups * 8 + 255) / 256;
  ++*L.launches;
  return launch_pdl(quantize_act_kernel, static_cast<unsigned>(blocks), 256, 0, L.stream, x, M, K, ldx, codes, scales,
                    dst_rows, fanout, M * fanout, pair_w, sorted_w);
}

}  // namespace qarl
