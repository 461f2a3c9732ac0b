// Small host helpers shared by the translation units that implement the C ABI.
#pragma once
#include <stdio.h>

#include <nvtx3/nvToolsExt.h>

#include "common.cuh"

namespace qarl {

// NVTX range around an entry point (visible in a timeline profiler; a pointer check when none is attached).
struct NvtxRange {
  explicit NvtxRange(const char* name) { nvtxRangePushA(name); }
  ~NvtxRange() { nvtxRangePop(); }
  NvtxRange(const NvtxRange&) = delete;
  NvtxRange& operator=(const NvtxRange&) = delete;
};

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

inline int cuda_fail(qarl_ctx* ctx, cudaError_t e, const char* where) {
  snprintf(ctx->err, sizeof(ctx->err), "%s: %s", where, cudaGetErrorString(e));
  return QARL_ERR_CUDA;
}

inline Launch make_launch(qarl_ctx* ctx, void* stream) {
  Launch L;
  L.stream = static_cast<cudaStream_t>(stream);
  L.device = ctx->device;
  L.sm_count = ctx->sm_count;
  L.d_status = ctx->d_status;
  L.launches = &ctx->launches;
  L.wait_limit_ns = ctx->wait_limit_ns;
  L.stop_after_stages = ctx->stop_after_stages;
  L.gemm_path = ctx->gemm_path;
  return L;
}

// Record a timing mark on the stream if stage timing is on and events are left.
inline void mark(qarl_ctx* ctx, cudaStream_t st, int stage) {
  if (ctx->marks_used >= ctx->marks.size()) return;
  if (cudaEventRecord(ctx->marks[ctx->marks_used], st) != cudaSuccess) return;
  ctx->mark_stage[ctx->marks_used++] = stage;
}

// The block-scaled FP8 GEMM with its error reporting.
inline int run_gemm(qarl_ctx* ctx, const Launch& L, const GemmArgs& a) {
  CUresult cu = CUDA_SUCCESS;
  cudaError_t e = launch_gemm(L, ctx->encode, a, &cu);
  if (cu != CUDA_SUCCESS) {
    snprintf(ctx->err, sizeof(ctx->err), "cuTensorMapEncodeTiled failed with CUresult %d", static_cast<int>(cu));
    return QARL_ERR_CUDA;
  }
  if (e != cudaSuccess) return cuda_fail(ctx, e, "gemm launch");
  return QARL_OK;
}

}  // namespace qarl
