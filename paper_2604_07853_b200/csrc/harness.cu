// Test-harness glue (not part of the quantized-forward API): a row-invariant RMSNorm used
// between layers by the alignment-stack test.
#include "common.cuh"
#include "../../include/qarl_harness.h"
#include "ptx_sm100.cuh"

namespace qarl {
namespace {

// One warp per row.  Lane l owns the 16-byte chunks l, l+32, l+64, ... of the row; its partial
// sum runs over them in ascending order, then a fixed xor-butterfly combines the 32 partials.
__global__ void __launch_bounds__(256) rmsnorm_kernel(const uint16_t* __restrict__ x, int64_t M, int64_t H, float eps,
                                                      uint16_t* __restrict__ out) {
  const int64_t row = (static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x) >> 5;
  if (row >= M) return;
  const int lane = threadIdx.x & 31;
  const uint4* src = reinterpret_cast<const uint4*>(x + row * H);
  const int chunks = static_cast<int>(H / 8);
  float ss = 0.0f;
  for (int c = lane; c < chunks; c += 32) {
    const uint4 v = src[c];
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const float a = bf16_bits_to_f32(w[i] & 0xFFFFu), b = bf16_bits_to_f32(w[i] >> 16);
      ss = __fmaf_rn(a, a, ss);
      ss = __fmaf_rn(b, b, ss);
    }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) ss = __fadd_rn(ss, __shfl_xor_sync(0xFFFFFFFFu, ss, o));
  const float r = rsqrtf(__fadd_rn(__fdiv_rn(ss, static_cast<float>(H)), eps));
  uint4* dst = reinterpret_cast<uint4*>(out + row * H);
  for (int c = lane; c < chunks; c += 32) {
    const uint4 v = src[c];
    uint4 o;
    o.x = pack_bf16x2(__fmul_rn(bf16_bits_to_f32(v.x & 0xFFFFu), r), __fmul_rn(bf16_bits_to_f32(v.x >> 16), r));
    o.y = pack_bf16x2(__fmul_rn(bf16_bits_to_f32(v.y & 0xFFFFu), r), __fmul_rn(bf16_bits_to_f32(v.y >> 16), r));
    o.z = pack_bf16x2(__fmul_rn(bf16_bits_to_f32(v.z & 0xFFFFu), r), __fmul_rn(bf16_bits_to_f32(v.z >> 16), r));
    o.w = pack_bf16x2(__fmul_rn(bf16_bits_to_f32(v.w & 0xFFFFu), r), __fmul_rn(bf16_bits_to_f32(v.w >> 16), r));
    dst[c] = o;
  }
}

// A wait that can never be satisfied, bounded like every wait in the GEMM pipeline.
__global__ void wait_selftest_kernel(unsigned long long limit_ns, int* status) {
  __shared__ uint64_t bar;
  if (threadIdx.x == 0) {
    ptx::mbar_init(&bar, 1);
    ptx::fence_mbar_init();
    if (!ptx::mbar_wait_bounded(&bar, 0, limit_ns)) set_status(status, QARL_ERR_DEVICE_TIMEOUT);
  }
}

}  // namespace

cudaError_t launch_wait_selftest(const Launch& L, unsigned long long limit_ns) {
  wait_selftest_kernel<<<1, 32, 0, L.stream>>>(limit_ns, L.d_status);
  ++*L.launches;
  return cudaGetLastError();
}

cudaError_t launch_rmsnorm(const Launch& L, const uint16_t* x, int64_t M, int64_t H, float eps, uint16_t* out) {
  if (M == 0) return cudaSuccess;
  const int64_t blocks = (M * 32 + 255) / 256;
  rmsnorm_kernel<<<static_cast<unsigned>(blocks), 256, 0, L.stream>>>(x, M, H, eps, out);
  ++*L.launches;
  return cudaGetLastError();
}

}  // namespace qarl
