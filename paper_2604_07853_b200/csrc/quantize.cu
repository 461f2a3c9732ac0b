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
                                                              float* __restrict__ scales,
                                                              uint8_t* __restrict__ pub_codes,
                                                              float* __restrict__ pub_scales) {
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
  if (tid == 0) {
    scales[blk] = s;
    if (pub_scales) pub_scales[blk] = s;
  }
#pragma unroll
  for (int p = 0; p < 4; ++p) {
    uint4 out;
    encode8(v[p][0], inv, out.x, out.y);
    encode8(v[p][1], inv, out.z, out.w);
    *reinterpret_cast<uint4*>(codes + base + static_cast<int64_t>(r0 + 32 * p) * K) = out;
    // the rollout engine's copy of the same tensors (Sec. 3.1 item 3), written from the same registers
    if (pub_codes) *reinterpret_cast<uint4*>(pub_codes + base + static_cast<int64_t>(r0 + 32 * p) * K) = out;
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


// ---- W4A16 weights (Sec. 2.2, integer quantization): W_q = clamp(round(W/s) + z, 0, 15) ------
// One (s, z) per 128 consecutive K elements of a weight row: lo = min(0, min W), hi = max(0, max W),
// s = bf16(max(hi - lo, 2^-40) / 15), z = clamp(rint(-lo / s), 0, 15).  8 threads per group, 16
// elements (two 32-bit words of codes) each.  Inside a word the eight codes e0..e7 sit in the
// nibble order e0 e2 e4 e6 e1 e3 e5 e7 (low nibble first), so that (word >> 4j) & 0x000F000F
// yields the adjacent pair (e_2j, e_2j+1) in the two halves of a register.  The words are
// stored tile-major: the codes of 128 weight rows x 64 K-elements form one contiguous 4 KB chunk
// (what one K-step of the GEMM consumes for one half tile, fetched by a single bulk copy), laid
// out inside as [word quad 0..1][row 0..127][16 bytes] so that the 128 threads that expand it
// read consecutive 16-byte pieces.  Scales (bf16 bits) and zero points are stored group-major,
// [E][K/128][N], contiguous along the weight rows.
// rint(w / s) + z clamped to 0..15 for one element, equal to the IEEE-division form bit for bit
// but without a division per element.  w and s are bf16 values (8 significant bits each), so the
// exact quotient is either exactly half-way between two integers or at least 2^-14 (relative) away
// from such a point: the product with inv = fl(1 / s) (relative error ~2^-23) then rounds to the
// same integer except at exact ties, which the exact residual r = w - q0 s identifies
// (2 r = +-s) and resolves to the even neighbour.
__device__ __forceinline__ uint32_t w4_code(float w, float s, float inv, float zm) {
  const float kMagic = 12582912.0f;               // 1.5 * 2^23: adding it rounds to an integer
  float q0 = __fsub_rn(__fmaf_rn(w, inv, kMagic), kMagic);
  const float r = __fmaf_rn(-q0, s, w);           // exact: q0 s has at most 13 significant bits
  if (fabsf(__fadd_rn(r, r)) == s) {              // tie between q0 and q0 + sign(r)
    const float other = r > 0.0f ? q0 + 1.0f : q0 - 1.0f;
    const float half = 0.5f * q0;
    if (__fsub_rn(__fadd_rn(half, kMagic), kMagic) != half) q0 = other;  // q0 odd: the other one is even
  }
  // zm = z + 2^23: the code is clamped in that domain, where the integer sits in the low mantissa bits
  const float v = fminf(fmaxf(__fadd_rn(q0, zm), 8388608.0f), 8388623.0f);
  return __float_as_uint(v) & 15u;
}

__device__ __forceinline__ uint32_t w4_word(const uint4& v, float s, float inv, float zm) {
  const uint32_t in[4] = {v.x, v.y, v.z, v.w};
  uint32_t word = 0;
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    word |= w4_code(bf16_bits_to_f32(in[j] & 0xFFFFu), s, inv, zm) << (4 * j);
    word |= w4_code(__uint_as_float(in[j] & 0xFFFF0000u), s, inv, zm) << (4 * j + 16);
  }
  return word;
}

// ---- FP4 (e2m1) weights (Sec. 2.2, floating-point quantization): s = amax / 6, W_q = [W / s]_FP4 ----
// Same groups, code order and storage as the integer format; s = bf16(max(amax, 2^-40) / 6).
// The magnitude code of |w| / s rounded to the nearest of 0, .5, 1, 1.5, 2, 3, 4, 6 (ties to the even
// code, saturating) is the number of rounding boundaries it passes: .25 .75 1.25 1.75 2.5 3.5 5, where a
// value exactly on a boundary goes to the neighbour with mantissa bit 0 (so the boundaries are
// exclusive, inclusive, exclusive, ...).  |w| / s against a boundary b compares like |w| against b s,
// and b s is exact in fp32 (3 x 8 significant bits), as is the comparison of the IEEE quotient:
// two distinct numbers of at most 8 and 11 bits differ by more than the quotient's rounding error.
struct Fp4Bounds { float t[7]; };
__device__ __forceinline__ Fp4Bounds fp4_bounds(float s) {
  Fp4Bounds b;
  const float k[7] = {0.25f, 0.75f, 1.25f, 1.75f, 2.5f, 3.5f, 5.0f};
#pragma unroll
  for (int i = 0; i < 7; ++i) b.t[i] = __fmul_rn(k[i], s);
  return b;
}
__device__ __forceinline__ uint32_t fp4_code(uint32_t bits_hi, const Fp4Bounds& b) {  // bf16 bits in [16, 32)
  const float a = __uint_as_float(bits_hi & 0x7FFF0000u);
  const uint32_t mag = (a > b.t[0]) + (a >= b.t[1]) + (a > b.t[2]) + (a >= b.t[3]) + (a > b.t[4]) + (a >= b.t[5]) +
                       (a > b.t[6]);
  return ((bits_hi >> 28) & 8u) | mag;
}
__device__ __forceinline__ uint32_t fp4_word(const uint4& v, const Fp4Bounds& b) {
  const uint32_t in[4] = {v.x, v.y, v.z, v.w};
  uint32_t word = 0;
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    word |= fp4_code(in[j] << 16, b) << (4 * j);
    word |= fp4_code(in[j] & 0xFFFF0000u, b) << (4 * j + 16);
  }
  return word;
}

__device__ __forceinline__ void minmax_u4(const uint4& v, float& lo, float& hi) {
  const uint32_t in[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    const float a = bf16_bits_to_f32(in[j] & 0xFFFFu), b = __uint_as_float(in[j] & 0xFFFF0000u);
    lo = fminf(lo, fminf(a, b));
    hi = fmaxf(hi, fmaxf(a, b));
  }
}

template <int FMT>  // 0: unsigned 4-bit integer with zero point, 1: e2m1 (no zero point: `zeros` unused)
__global__ void __launch_bounds__(256) quantize_weight_w4_kernel(const uint16_t* __restrict__ w, int64_t rows,
                                                                 int64_t N, int64_t K,
                                                                 uint8_t* __restrict__ packed,
                                                                 uint16_t* __restrict__ scales,
                                                                 uint8_t* __restrict__ zeros,
                                                                 uint8_t* __restrict__ pub_packed,
                                                                 uint16_t* __restrict__ pub_scales,
                                                                 uint8_t* __restrict__ pub_zeros) {
  pdl_trigger();
  pdl_wait();
  // 32-bit index arithmetic (the launcher guarantees fewer than 2^31 groups): 64-bit divisions
  // would cost more instructions than the quantization itself
  const uint32_t kb = static_cast<uint32_t>(K / kBlock);
  const uint32_t gid = (blockIdx.x * blockDim.x + threadIdx.x) >> 3;
  const bool live = gid < static_cast<uint32_t>(rows) * kb;
  const uint32_t gg = live ? gid : 0u;
  const uint32_t row32 = gg / kb, g32 = gg - row32 * kb;
  const int64_t row = row32, g = g32;
  const int sub = threadIdx.x & 7;
  const uint4* src = reinterpret_cast<const uint4*>(w + row * K + g * kBlock + sub * 16);
  uint4 v0 = make_uint4(0, 0, 0, 0), v1 = v0;
  if (live) {
    v0 = __ldg(src);
    v1 = __ldg(src + 1);
  }
  float lo = 0.0f, hi = 0.0f;
  minmax_u4(v0, lo, hi);
  minmax_u4(v1, lo, hi);
#pragma unroll
  for (int o = 4; o > 0; o >>= 1) {
    lo = fminf(lo, __shfl_xor_sync(0xFFFFFFFFu, lo, o));
    hi = fmaxf(hi, __shfl_xor_sync(0xFFFFFFFFu, hi, o));
  }
  uint32_t s_bits;
  float zf = 0.0f;
  uint2 out;
  if constexpr (FMT == 0) {
    const float range = fmaxf(__fsub_rn(hi, lo), kAmaxFloor);
    s_bits = f32_to_bf16_bits(__fdiv_rn(range, 15.0f));
    const float s = bf16_bits_to_f32(s_bits);
    zf = fminf(fmaxf(rintf(__fdiv_rn(-lo, s)), 0.0f), 15.0f);
    const float inv = __fdiv_rn(1.0f, s);
    const float zm = zf + 8388608.0f;
    out = make_uint2(w4_word(v0, s, inv, zm), w4_word(v1, s, inv, zm));
  } else {
    const float amax = fmaxf(fmaxf(-lo, hi), kAmaxFloor);  // lo <= 0 <= hi
    s_bits = f32_to_bf16_bits(__fdiv_rn(amax, 6.0f));
    const Fp4Bounds b = fp4_bounds(bf16_bits_to_f32(s_bits));
    out = make_uint2(fp4_word(v0, b), fp4_word(v1, b));
  }
  if (!live) return;
  const uint32_t e32 = row32 / static_cast<uint32_t>(N);
  const int64_t e = e32, n = row32 - e32 * static_cast<uint32_t>(N);
  {
    const int64_t ks = g * 2 + (sub >> 2);  // K-step of 64 elements
    const int64_t chunk = (e * (N / kBlock) + (n >> 7)) * (K / 64) + ks;
    const int quad = (sub & 3) >> 1, piece = sub & 1;  // words 2(sub%4), 2(sub%4)+1 of the K-step's eight
    const int64_t at = chunk * 4096 + quad * 2048 + (n & (kBlock - 1)) * 16 + piece * 8;
    *reinterpret_cast<uint2*>(packed + at) = out;
    if (pub_packed) *reinterpret_cast<uint2*>(pub_packed + at) = out;  // the rollout engine's copy (Sec. 3.1 item 3)
  }
  if (sub == 0) {
    const int64_t idx = (e * kb + g) * N + n;
    scales[idx] = static_cast<uint16_t>(s_bits);
    if (FMT == 0) zeros[idx] = static_cast<uint8_t>(zf);
    if (pub_packed) {
      pub_scales[idx] = static_cast<uint16_t>(s_bits);
      if (FMT == 0) pub_zeros[idx] = static_cast<uint8_t>(zf);
    }
  }
}

// Copies bf16 row t of x to the `fanout` rows dst_rows[t*fanout + j] of out (expert-sorted
// order) and scatters the pair weights alongside; 16 bytes per thread.
__global__ void __launch_bounds__(256) scatter_rows_kernel(const uint16_t* __restrict__ x, int64_t M, int64_t H,
                                                           uint16_t* __restrict__ out,
                                                           const int32_t* __restrict__ dst_rows, int fanout,
                                                           int64_t dst_rows_total,
                                                           const float* __restrict__ pair_w,
                                                           float* __restrict__ sorted_w) {
  pdl_trigger();
  pdl_wait();
  const int64_t per_row = H / 8;
  const int64_t idx = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (idx >= M * per_row) return;
  const int64_t row = idx / per_row, c = idx % per_row;
  const uint4 v = __ldg(reinterpret_cast<const uint4*>(x + row * H) + c);
  for (int j = 0; j < fanout; ++j) {
    const int64_t d = min(max(static_cast<int64_t>(dst_rows[row * fanout + j]), int64_t(0)), dst_rows_total - 1);
    reinterpret_cast<uint4*>(out + d * H)[c] = v;
    if (c == 0 && sorted_w != nullptr) sorted_w[d] = pair_w[row * fanout + j];
  }
}

}  // namespace

cudaError_t launch_quantize_weight(const Launch& L, const uint16_t* w, int64_t E, int64_t N, int64_t K,
                                   uint8_t* codes, float* scales, uint8_t* pub_codes, float* pub_scales) {
  const int64_t blocks = E * (N / kBlock) * (K / kBlock);
  if (blocks == 0) return cudaSuccess;
  ++*L.launches;
  return launch_pdl(quantize_weight_kernel, static_cast<unsigned>(blocks), 256, 0, L.stream, w, N, K, codes, scales,
                    pub_codes, pub_scales);
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

cudaError_t launch_quantize_weight_w4(const Launch& L, int fmt, const uint16_t* w, int64_t E, int64_t N, int64_t K,
                                      uint8_t* packed, uint16_t* scales, uint8_t* zeros, uint8_t* pub_packed,
                                      uint16_t* pub_scales, uint8_t* pub_zeros) {
  const int64_t groups = E * N * (K / kBlock);
  if (groups == 0) return cudaSuccess;
  const int64_t blocks = (groups * 8 + 255) / 256;
  ++*L.launches;
  return launch_pdl(fmt == kFmtE2m1 ? quantize_weight_w4_kernel<1> : quantize_weight_w4_kernel<0>,
                    static_cast<unsigned>(blocks), 256, 0, L.stream, w, E * N, N, K, packed, scales, zeros, pub_packed,
                    pub_scales, pub_zeros);
}

cudaError_t launch_scatter_rows(const Launch& L, const uint16_t* x, int64_t M, int64_t H, uint16_t* out,
                                const int32_t* dst_rows, int fanout, const float* pair_w, float* sorted_w) {
  const int64_t threads = M * (H / 8);
  if (threads == 0) return cudaSuccess;
  ++*L.launches;
  return launch_pdl(scatter_rows_kernel, static_cast<unsigned>((threads + 255) / 256), 256, 0, L.stream, x, M, H, out,
                    dst_rows, fanout, M * fanout, pair_w, sorted_w);
}

}  // namespace qarl
