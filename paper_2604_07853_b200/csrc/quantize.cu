// Block quantizers (Sec. 2.2, floating-point quantization): per block amax -> s = amax/448 ->
// e4m3 codes, for 128x128 weight blocks and 1x128 activation groups.  Both kernels are
// HBM-bound: 128-bit loads, 128-bit stores, every input byte read once.
#include "common.cuh"
#include "quant_device.cuh"

namespace qarl {
namespace {

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
__device__ __forceinline__ __nv_bfloat162 as_bf2(uint32_t u) { return *reinterpret_cast<__nv_bfloat162*>(&u); }
__device__ __forceinline__ uint32_t bf2_bits(__nv_bfloat162 v) { return *reinterpret_cast<uint32_t*>(&v); }

__device__ __forceinline__ uint32_t fma_bf2(uint32_t a, uint32_t b, uint32_t c) {
  uint32_t d;
  asm("fma.rn.bf16x2 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
  return d;
}
__device__ __forceinline__ uint32_t add_bf2(uint32_t a, uint32_t b) {
  uint32_t d;
  asm("add.rn.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
  return d;
}
// Whether a boundary was passed is read from a sign bit, with integer instructions only.  d is the
// bf16x2 difference value - boundary (never a subnormal: the operands have few bits).  Adding 0x0080 to
// each half (one exponent step) makes +0 positive and keeps every other sign: sign clear <=> d >= 0, for
// boundaries that belong to the upper code.  Subtracting it makes +0 negative and keeps every other sign
// (a borrow out of the low half can only turn a high half that is +0 or positive-minimal around, and the
// latter cannot occur): sign clear <=> d > 0, for boundaries that belong to the lower code.
constexpr uint32_t kTieUp = 0x00800080u, kTieDown = 0xFF7FFF80u, kSigns = 0x80008000u;

// q = clamp(rint(w / s) + z, 0, 15) for two adjacent elements at once, equal to the IEEE-division form
// bit for bit but without a division: q is the number of boundaries (j - z - 1/2) s, j = 1..15, that w
// passes, where a w exactly on a boundary goes to the even neighbour of rint.  w and s are bf16 (8
// significant bits), the multiplier m = j - z - 1/2 has at most 6, so w - m s is exact before the one
// rounding of a fused multiply-add, which keeps its sign and gives zero only for an exact tie, also in
// bf16; and the IEEE quotient w / s compares with m as w does with m s, because distinct numbers of 8 and
// 14 bits differ by far more than the quotient's rounding error.  A four-level binary search over j
// (8, then +-4, +-2, +-1) therefore yields the four bits of q, one bf16x2 FMA per level.
// Ties: the boundary below code j belongs to rint value j - 1 - z; it goes up when that is odd, i.e.
// for even j when z is even and for odd j when z is odd.
struct W4Group {
  uint32_t neg_s;         // -s twice
  uint32_t m8;            // 7.5 - z twice: the first boundary
  uint32_t tie_hi, tie_lo;  // kTieUp / kTieDown for the first three levels (even j) / the last level (odd j)
};
__device__ __forceinline__ W4Group w4_group(uint32_t s_bits, float zf) {
  W4Group g;
  g.neg_s = (s_bits | 0x8000u) * 0x00010001u;
  g.m8 = f32_to_bf16_bits(7.5f - zf) * 0x00010001u;   // a half-integer below 16: exact
  const bool z_odd = (static_cast<int>(zf) & 1) != 0;
  g.tie_hi = z_odd ? kTieDown : kTieUp;
  g.tie_lo = z_odd ? kTieUp : kTieDown;
  return g;
}
// codes of the pair (elements 2j, 2j+1 of a word's eight) OR-ed into `word` at bits [4j, 4j+4) and [16+4j, 20+4j)
template <int J>
__device__ __forceinline__ uint32_t w4_codes2(uint32_t word, uint32_t w2, const W4Group& g) {
  uint32_t m = g.m8;
  uint32_t t = fma_bf2(m, g.neg_s, w2) + g.tie_hi;                       // j = 8
  word |= (~t >> (12 - 4 * J)) & (0x00080008u << (4 * J));
  m = add_bf2(m, 0xC080C080u ^ (~t & kSigns));                           // +4 where passed, else -4
  t = fma_bf2(m, g.neg_s, w2) + g.tie_hi;
  word |= (~t >> (13 - 4 * J)) & (0x00040004u << (4 * J));
  m = add_bf2(m, 0xC000C000u ^ (~t & kSigns));                           // +-2
  t = fma_bf2(m, g.neg_s, w2) + g.tie_hi;
  word |= (~t >> (14 - 4 * J)) & (0x00020002u << (4 * J));
  m = add_bf2(m, 0xBF80BF80u ^ (~t & kSigns));                           // +-1
  t = fma_bf2(m, g.neg_s, w2) + g.tie_lo;
  word |= (~t >> (15 - 4 * J)) & (0x00010001u << (4 * J));
  return word;
}
__device__ __forceinline__ uint32_t w4_word(const uint4& v, const W4Group& g) {
  return w4_codes2<3>(w4_codes2<2>(w4_codes2<1>(w4_codes2<0>(0u, v.x, g), v.y, g), v.z, g), v.w, g);
}

// ---- FP4 (e2m1) weights (Sec. 2.2, floating-point quantization): s = amax / 6, W_q = [W / s]_FP4 ----
// Same groups, code order and storage as the integer format; s = bf16(max(amax, 2^-40) / 6).
// The magnitude code of |w| / s rounded to the nearest of 0, .5, 1, 1.5, 2, 3, 4, 6 (ties to the even
// code, saturating) is the number of rounding boundaries b = .25 .75 1.25 1.75 2.5 3.5 5 it passes, where a
// value exactly on a boundary goes to the neighbour with mantissa bit 0 (so the boundaries are
// exclusive, inclusive, exclusive, ...).  As above, the sign of |w| - b s from one bf16x2 FMA decides
// each comparison exactly.  Three levels give the three bits: b = 1.75 (>=); then 3.5 or .75 (>=); then 5,
// 2.5, 1.25 or .25 (>).  With P1, P2 = +-1 for passed / not passed, the next boundaries are the exact
// bf16 polynomials  b1 = 2.125 + 1.375 P1  and  b0 = (2.25 + 1.5 P1) + P2 (.875 + .375 P1),  kept negated.
template <int J>
__device__ __forceinline__ uint32_t fp4_codes2(uint32_t word, uint32_t w2, uint32_t s2) {
  const uint32_t a2 = w2 & 0x7FFF7FFFu;
  uint32_t t = fma_bf2(0xBFE0BFE0u /* -1.75 */, s2, a2) + kTieUp;
  word |= (~t >> (13 - 4 * J)) & (0x00040004u << (4 * J));
  const uint32_t p1 = 0x3F803F80u | (t & kSigns);                        // +1 where passed, else -1
  const uint32_t nb1 = fma_bf2(p1, 0xBFB0BFB0u /* -1.375 */, 0xC008C008u /* -2.125 */);
  t = fma_bf2(nb1, s2, a2) + kTieUp;
  word |= (~t >> (14 - 4 * J)) & (0x00020002u << (4 * J));
  const uint32_t p2 = 0x3F803F80u | (t & kSigns);
  const uint32_t u = fma_bf2(p1, 0xBFC0BFC0u /* -1.5 */, 0xC010C010u /* -2.25 */);
  const uint32_t v = fma_bf2(p1, 0xBEC0BEC0u /* -.375 */, 0xBF60BF60u /* -.875 */);
  t = fma_bf2(fma_bf2(p2, v, u), s2, a2) + kTieDown;
  word |= (~t >> (15 - 4 * J)) & (0x00010001u << (4 * J));
  if (J == 3) word |= w2 & 0x80008000u;                                  // sign: bit 3 of the code
  else word |= (w2 >> (12 - 4 * J)) & (0x00080008u << (4 * J));
  return word;
}
__device__ __forceinline__ uint32_t fp4_word(const uint4& v, uint32_t s2) {
  return fp4_codes2<3>(fp4_codes2<2>(fp4_codes2<1>(fp4_codes2<0>(0u, v.x, s2), v.y, s2), v.z, s2), v.w, s2);
}
__device__ __forceinline__ __nv_bfloat162 absmax_u4(const uint4& v, __nv_bfloat162 m) {
  m = __hmax2(m, as_bf2(v.x & 0x7FFF7FFFu));
  m = __hmax2(m, as_bf2(v.y & 0x7FFF7FFFu));
  m = __hmax2(m, as_bf2(v.z & 0x7FFF7FFFu));
  return __hmax2(m, as_bf2(v.w & 0x7FFF7FFFu));
}

__device__ __forceinline__ void minmax_u4(const uint4& v, __nv_bfloat162& lo, __nv_bfloat162& hi) {
  const uint32_t in[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    lo = __hmin2(lo, as_bf2(in[j]));
    hi = __hmax2(hi, as_bf2(in[j]));
  }
}

// A block owns 32 consecutive weight rows (8 threads per row, 16 elements each) and walks a range of
// their K-groups, so that the row and chunk arithmetic is done once and the next group's 32 bytes are
// in flight while the current one is encoded.  Rows never straddle an expert (N % 128 == 0).
template <int FMT>  // 0: unsigned 4-bit integer with zero point, 1: e2m1 (no zero point: `zeros` unused)
__global__ void __launch_bounds__(256) quantize_weight_w4_kernel(const uint16_t* __restrict__ w, int64_t N, int64_t K,
                                                                 int groups_per_block,
                                                                 uint8_t* __restrict__ packed,
                                                                 uint16_t* __restrict__ scales,
                                                                 uint8_t* __restrict__ zeros,
                                                                 uint8_t* __restrict__ pub_packed,
                                                                 uint16_t* __restrict__ pub_scales,
                                                                 uint8_t* __restrict__ pub_zeros) {
  pdl_trigger();
  pdl_wait();
  const int kb = static_cast<int>(K / kBlock);
  const int g_begin = blockIdx.y * groups_per_block, g_end = min(kb, g_begin + groups_per_block);
  const uint32_t row = blockIdx.x * 32u + (threadIdx.x >> 3);   // over all experts
  const int sub = threadIdx.x & 7;
  const uint32_t e = row / static_cast<uint32_t>(N), n = row - e * static_cast<uint32_t>(N);
  const uint4* src = reinterpret_cast<const uint4*>(w + static_cast<int64_t>(row) * K + sub * 16) + g_begin * 16;
  // byte offset of this thread's two words in the chunk of K-step 2g + sub/4: words 2(sub%4), 2(sub%4)+1
  const int64_t chunk0 = (static_cast<int64_t>(e) * (N / kBlock) + (n >> 7)) * (K / 64) + (sub >> 2);
  int64_t at = (chunk0 + 2 * g_begin) * 4096 + ((sub & 3) >> 1) * 2048 + (n & (kBlock - 1)) * 16 + (sub & 1) * 8;
  int64_t idx = (static_cast<int64_t>(e) * kb + g_begin) * N + n;
  if (g_begin >= g_end) return;
  uint4 v0 = __ldg(src), v1 = __ldg(src + 1);
  for (int g = g_begin; g < g_end; ++g, src += 16, at += 8192, idx += N) {
    const uint4 c0 = v0, c1 = v1;
    if (g + 1 < g_end) {
      v0 = __ldg(src + 16);
      v1 = __ldg(src + 17);
    }
    uint32_t s_bits;
    float zf = 0.0f;
    uint2 out;
    if constexpr (FMT == 0) {
      __nv_bfloat162 lo2 = as_bf2(0u), hi2 = as_bf2(0u);  // zero stays representable: lo <= 0 <= hi
      minmax_u4(c0, lo2, hi2);
      minmax_u4(c1, lo2, hi2);
#pragma unroll
      for (int o = 4; o > 0; o >>= 1) {
        lo2 = __hmin2(lo2, as_bf2(__shfl_xor_sync(0xFFFFFFFFu, bf2_bits(lo2), o)));
        hi2 = __hmax2(hi2, as_bf2(__shfl_xor_sync(0xFFFFFFFFu, bf2_bits(hi2), o)));
      }
      const float lo = fminf(__low2float(lo2), __high2float(lo2)), hi = fmaxf(__low2float(hi2), __high2float(hi2));
      const float range = fmaxf(__fsub_rn(hi, lo), kAmaxFloor);
      s_bits = f32_to_bf16_bits(__fdiv_rn(range, 15.0f));
      const float s = bf16_bits_to_f32(s_bits);
      zf = fminf(fmaxf(rintf(__fdiv_rn(-lo, s)), 0.0f), 15.0f);
      const W4Group grp = w4_group(s_bits, zf);
      out = make_uint2(w4_word(c0, grp), w4_word(c1, grp));
    } else {
      __nv_bfloat162 m2 = absmax_u4(c1, absmax_u4(c0, as_bf2(0u)));
#pragma unroll
      for (int o = 4; o > 0; o >>= 1) m2 = __hmax2(m2, as_bf2(__shfl_xor_sync(0xFFFFFFFFu, bf2_bits(m2), o)));
      const float amax = fmaxf(fmaxf(__low2float(m2), __high2float(m2)), kAmaxFloor);
      s_bits = f32_to_bf16_bits(__fdiv_rn(amax, 6.0f));
      const uint32_t s2 = s_bits * 0x00010001u;
      out = make_uint2(fp4_word(c0, s2), fp4_word(c1, s2));
    }
    *reinterpret_cast<uint2*>(packed + at) = out;
    if (pub_packed) *reinterpret_cast<uint2*>(pub_packed + at) = out;  // the rollout engine's copy (Sec. 3.1 item 3)
    if (sub == 0) {
      scales[idx] = static_cast<uint16_t>(s_bits);
      if (FMT == 0) zeros[idx] = static_cast<uint8_t>(zf);
      if (pub_packed) {
        pub_scales[idx] = static_cast<uint16_t>(s_bits);
        if (FMT == 0) pub_zeros[idx] = static_cast<uint8_t>(zf);
      }
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
  const int64_t row_blocks = E * N / 32, kb = K / kBlock;
  if (row_blocks == 0 || kb == 0) return cudaSuccess;
  // split the K-groups of a row block over several CTAs until the grid fills the device a few times over
  const int64_t want = static_cast<int64_t>(L.sm_count) * 32;
  const int64_t split = std::min<int64_t>(kb, std::max<int64_t>(1, (want + row_blocks - 1) / row_blocks));
  const int per = static_cast<int>((kb + split - 1) / split);
  const dim3 grid(static_cast<unsigned>(row_blocks), static_cast<unsigned>((kb + per - 1) / per));
  ++*L.launches;
  return launch_pdl(fmt == kFmtE2m1 ? quantize_weight_w4_kernel<1> : quantize_weight_w4_kernel<0>, grid, 256, 0,
                    L.stream, w, N, K, per, packed, scales, zeros, pub_packed, pub_scales, pub_zeros);
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
