// Element-wise kernels of the MoE layer's full-precision backward (Sec. 3.1 item 2; the GEMMs are
// in gemm_bf16_sm100.cu).  All HBM-bound, 16-byte accesses, one fixed order of arithmetic.
#include <math.h>

#include "common.cuh"

namespace qarl {
namespace {

__device__ __forceinline__ uint32_t bf16x2(float lo, float hi) {
  const __nv_bfloat162 b = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<const uint32_t*>(&b);
}

// dy[pos(t, j)] = bf16( w[t, j] * dout[t] ): the gradient of the combine, written in expert-sorted
// order.  One thread per 8 columns of a token row; the row is read once and written k times.
__global__ void __launch_bounds__(256) scatter_scale_rows_kernel(const uint16_t* __restrict__ dout, int64_t M, int64_t H,
                                                                 uint16_t* __restrict__ dy,
                                                                 const int32_t* __restrict__ dst_rows, int fanout,
                                                                 int64_t dst_rows_total,
                                                                 const float* __restrict__ pair_w) {
  pdl_trigger();
  pdl_wait();
  const int64_t per_row = H / 8;
  const int64_t idx = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (idx >= M * per_row) return;
  const int64_t row = idx / per_row, c = idx % per_row;
  const uint4 v = __ldg(reinterpret_cast<const uint4*>(dout + row * H) + c);
  const uint32_t in[4] = {v.x, v.y, v.z, v.w};
  for (int j = 0; j < fanout; ++j) {
    const float w = pair_w[row * fanout + j];
    const int64_t d = min(max(static_cast<int64_t>(dst_rows[row * fanout + j]), int64_t(0)), dst_rows_total - 1);
    uint32_t o[4];
#pragma unroll
    for (int q = 0; q < 4; ++q)
      o[q] = bf16x2(__fmul_rn(w, bf16_bits_to_f32(in[q] & 0xFFFFu)), __fmul_rn(w, __uint_as_float(in[q] & 0xFFFF0000u)));
    reinterpret_cast<uint4*>(dy + d * H)[c] = make_uint4(o[0], o[1], o[2], o[3]);
  }
}

// dG = dH u s (1 + g (1 - s)), dU = dH g s with s = 1 / (1 + exp(-g)), on the bf16 gate / up the
// forward saved; fp32 arithmetic, results rounded to bf16.  One thread per 8 columns.
__global__ void __launch_bounds__(256) swiglu_bwd_kernel(const uint16_t* __restrict__ gate_up,
                                                         const uint16_t* __restrict__ dh, int64_t P, int64_t I,
                                                         uint16_t* __restrict__ dgu) {
  pdl_trigger();
  pdl_wait();
  const int64_t per_row = I / 8;
  const int64_t idx = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (idx >= P * per_row) return;
  const int64_t row = idx / per_row, c = idx % per_row;
  const uint4 g4 = __ldg(reinterpret_cast<const uint4*>(gate_up + row * 2 * I) + c);
  const uint4 u4 = __ldg(reinterpret_cast<const uint4*>(gate_up + row * 2 * I + I) + c);
  const uint4 d4 = __ldg(reinterpret_cast<const uint4*>(dh + row * I) + c);
  const uint32_t gw[4] = {g4.x, g4.y, g4.z, g4.w}, uw[4] = {u4.x, u4.y, u4.z, u4.w}, dw[4] = {d4.x, d4.y, d4.z, d4.w};
  uint32_t og[4], ou[4];
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    float dg[2], du[2];
#pragma unroll
    for (int hsel = 0; hsel < 2; ++hsel) {
      const float g = hsel ? __uint_as_float(gw[q] & 0xFFFF0000u) : bf16_bits_to_f32(gw[q] & 0xFFFFu);
      const float u = hsel ? __uint_as_float(uw[q] & 0xFFFF0000u) : bf16_bits_to_f32(uw[q] & 0xFFFFu);
      const float d = hsel ? __uint_as_float(dw[q] & 0xFFFF0000u) : bf16_bits_to_f32(dw[q] & 0xFFFFu);
      const float s = 1.0f / (1.0f + expf(-g));
      dg[hsel] = d * u * s * (1.0f + g * (1.0f - s));
      du[hsel] = d * g * s;
    }
    og[q] = bf16x2(dg[0], dg[1]);
    ou[q] = bf16x2(du[0], du[1]);
  }
  reinterpret_cast<uint4*>(dgu + row * 2 * I)[c] = make_uint4(og[0], og[1], og[2], og[3]);
  reinterpret_cast<uint4*>(dgu + row * 2 * I + I)[c] = make_uint4(ou[0], ou[1], ou[2], ou[3]);
}

// Gradient of a routing weight: dwts[pair] = <dout[token], y[q]> with y the fp32 output of the down
// projection at sorted position q.  One warp per sorted row; lane-strided fp32 partial sums, then a
// shuffle tree: one fixed order.
__global__ void __launch_bounds__(256) pair_dot_kernel(const uint16_t* __restrict__ dout, const float* __restrict__ y,
                                                       const int32_t* __restrict__ sorted_pair, int64_t P, int64_t H,
                                                       int k, float* __restrict__ dwts) {
  pdl_trigger();
  pdl_wait();
  const int lane = threadIdx.x & 31;
  const int64_t q = (static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x) >> 5;
  if (q >= P) return;
  const int64_t pair = min(max(static_cast<int64_t>(sorted_pair[q]), int64_t(0)), P - 1);
  const uint16_t* drow = dout + (pair / k) * H;
  const float* yrow = y + q * H;
  float acc = 0.0f;
  for (int64_t c = lane * 4; c < H; c += 128) {
    const uint2 dv = __ldg(reinterpret_cast<const uint2*>(drow + c));
    const float4 yv = __ldg(reinterpret_cast<const float4*>(yrow + c));
    acc = __fmaf_rn(bf16_bits_to_f32(dv.x & 0xFFFFu), yv.x, acc);
    acc = __fmaf_rn(__uint_as_float(dv.x & 0xFFFF0000u), yv.y, acc);
    acc = __fmaf_rn(bf16_bits_to_f32(dv.y & 0xFFFFu), yv.z, acc);
    acc = __fmaf_rn(__uint_as_float(dv.y & 0xFFFF0000u), yv.w, acc);
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xFFFFFFFFu, acc, o);
  if (lane == 0) dwts[pair] = acc;
}

}  // namespace

cudaError_t launch_scatter_scale_rows(const Launch& L, const uint16_t* dout, int64_t M, int64_t H, uint16_t* dy,
                                      const int32_t* dst_rows, int fanout, const float* pair_w) {
  const int64_t threads = M * (H / 8);
  if (threads == 0) return cudaSuccess;
  ++*L.launches;
  return launch_pdl(scatter_scale_rows_kernel, static_cast<unsigned>((threads + 255) / 256), 256, 0, L.stream, dout, M, H,
                    dy, dst_rows, fanout, M * fanout, pair_w);
}

cudaError_t launch_swiglu_bwd(const Launch& L, const uint16_t* gate_up, const uint16_t* dh, int64_t P, int64_t I,
                              uint16_t* dgu) {
  const int64_t threads = P * (I / 8);
  if (threads == 0) return cudaSuccess;
  ++*L.launches;
  return launch_pdl(swiglu_bwd_kernel, static_cast<unsigned>((threads + 255) / 256), 256, 0, L.stream, gate_up, dh, P, I,
                    dgu);
}

cudaError_t launch_pair_dot(const Launch& L, const uint16_t* dout, const float* y, const int32_t* sorted_pair,
                            int64_t P, int64_t H, int64_t k, float* dwts) {
  if (P == 0) return cudaSuccess;
  ++*L.launches;
  return launch_pdl(pair_dot_kernel, static_cast<unsigned>((P * 32 + 255) / 256), 256, 0, L.stream, dout, y, sorted_pair,
                    P, H, static_cast<int>(k), dwts);
}

}  // namespace qarl
