// qarl_linear_fwd_static: the dense block-scaled projection for callers that may not allocate
// device memory at all.  The scratch qarl_linear_fwd takes from the caller (the quantized copy
// of the activations) lives here in a fixed device array that every GPU loading the library
// carries until the process exits.
#include <stdio.h>

#include <atomic>

#include "common.cuh"

namespace {

using namespace qarl;

// codes [M, K] (1 byte per element) followed by scales [M, K/128] (4 bytes per 128 elements)
constexpr size_t kCodesBytes = static_cast<size_t>(QARL_STATIC_LINEAR_MAX_ELEMS);
constexpr size_t kScalesBytes = kCodesBytes / 128 * sizeof(float);
constexpr size_t kScratchBytes = kCodesBytes + kScalesBytes;

// In host code this name is only a stand-in for the device array, never a device address;
// the address a kernel can use comes from cudaGetSymbolAddress (below), once per device.
static __device__ __align__(256) unsigned char g_static_scratch[kScratchBytes];

constexpr int kMaxDevices = 64;
// per device, written once; atomic because contexts on several host threads may make their first call at
// the same time (both resolve the same address)
std::atomic<unsigned char*> g_scratch_addr[kMaxDevices];

}  // namespace

extern "C" int qarl_linear_fwd_static(qarl_ctx* ctx, const void* x, int64_t M, int64_t K, const uint8_t* wc,
                                      const float* ws, int64_t N, void* y, void* stream) {
  if (!ctx || M < 0 || K <= 0 || N <= 0) return QARL_ERR_INVALID_ARG;
  if (N % kBlock || K % kBlock || N > 0x7FFFFF00ll) return QARL_ERR_UNSUPPORTED_SHAPE;
  if (M == 0) return QARL_OK;
  if (M > static_cast<int64_t>(kCodesBytes) / K) {
    snprintf(ctx->err, sizeof(ctx->err),
             "qarl_linear_fwd_static: M*K = %lld exceeds the built-in scratch of %lld elements; "
             "use qarl_linear_fwd with a caller workspace",
             static_cast<long long>(M * K), static_cast<long long>(QARL_STATIC_LINEAR_MAX_ELEMS));
    return QARL_ERR_UNSUPPORTED_SHAPE;
  }
  if (!x || !wc || !ws || !y) return QARL_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(x) & 15u) || (reinterpret_cast<uintptr_t>(wc) & 15u) ||
      (reinterpret_cast<uintptr_t>(y) & 15u) || (reinterpret_cast<uintptr_t>(ws) & 3u))
    return QARL_ERR_MISALIGNED;
  if (ctx->device < 0 || ctx->device >= kMaxDevices) return QARL_ERR_UNSUPPORTED_DEVICE;

  // Set-up on the first call for this device: resolve the array's device address while the
  // context's device is current.  (No allocation happens here or anywhere below.)
  if (g_scratch_addr[ctx->device].load(std::memory_order_acquire) == nullptr) {
    int cur = -1;
    cudaError_t e = cudaGetDevice(&cur);
    if (e != cudaSuccess || cur != ctx->device) {
      snprintf(ctx->err, sizeof(ctx->err), "qarl_linear_fwd_static: the context's device (%d) must be current",
               ctx->device);
      return e != cudaSuccess ? QARL_ERR_CUDA : QARL_ERR_INVALID_ARG;
    }
    unsigned char* p = nullptr;
    e = cudaGetSymbolAddress(reinterpret_cast<void**>(&p), g_static_scratch);
    if (e != cudaSuccess || p == nullptr) {
      snprintf(ctx->err, sizeof(ctx->err), "cudaGetSymbolAddress: %s", cudaGetErrorString(e));
      return QARL_ERR_CUDA;
    }
    g_scratch_addr[ctx->device].store(p, std::memory_order_release);
  }
  unsigned char* base = g_scratch_addr[ctx->device].load(std::memory_order_acquire);
  uint8_t* xc = base;
  float* xs = reinterpret_cast<float*>(base + kCodesBytes);

  Launch L;
  L.stream = static_cast<cudaStream_t>(stream);
  L.device = ctx->device;
  L.sm_count = ctx->sm_count;
  L.d_status = ctx->d_status;
  L.launches = &ctx->launches;
  // Every code and scale the GEMM reads for rows 0..M-1 is rewritten by this quantization, so
  // nothing left over from an earlier call (which the array keeps) is ever consumed and
  // nothing has to be cleared.
  cudaError_t e = launch_quantize_act(L, static_cast<const uint16_t*>(x), M, K, K, xc, xs, nullptr, 1);
  if (e != cudaSuccess) {
    snprintf(ctx->err, sizeof(ctx->err), "quantize_act: %s", cudaGetErrorString(e));
    return QARL_ERR_CUDA;
  }
  GemmArgs a{};
  a.mode = kModeLinear;
  a.a_codes = xc;
  a.a_scales = xs;
  a.rows_total = M;
  a.K = K;
  a.b_codes = wc;
  a.b_scales = ws;
  a.N = N;
  a.E = 1;
  a.out_bf16 = static_cast<uint16_t*>(y);
  CUresult cu = CUDA_SUCCESS;
  e = launch_gemm(L, ctx->encode, a, &cu);
  if (cu != CUDA_SUCCESS) {
    snprintf(ctx->err, sizeof(ctx->err), "cuTensorMapEncodeTiled failed with CUresult %d", static_cast<int>(cu));
    return QARL_ERR_CUDA;
  }
  if (e != cudaSuccess) {
    snprintf(ctx->err, sizeof(ctx->err), "gemm launch: %s", cudaGetErrorString(e));
    return QARL_ERR_CUDA;
  }
  return QARL_OK;
}
