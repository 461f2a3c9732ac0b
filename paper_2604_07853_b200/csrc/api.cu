// C ABI entry points: argument checks, workspace planning, kernel sequencing.  Nothing here
// allocates device memory except qarl_create (the 4-byte status word).
#include <stdio.h>
#include <string.h>

#include <new>
#include <vector>

#include "common.cuh"
#include "../../include/qarl_harness.h"

#include "api_util.cuh"

namespace {

using namespace qarl;

// Workspace carve-up of qarl_moe_fwd; every slice starts on a 256-byte boundary.
struct MoePlan {
  size_t chunk_hist, offsets, sorted_pair, pos_of_pair, sorted_w, a_codes, a_scales, h_codes, h_scales, contrib, sync, total;
};
MoePlan plan_moe(int64_t M, int64_t H, int64_t I, int64_t E, int64_t k) {
  const size_t P = static_cast<size_t>(M * k);
  MoePlan p{};
  size_t o = 0;
  auto take = [&](size_t bytes) {
    const size_t at = o;
    o = align_up(o + bytes, 256);
    return at;
  };
  p.chunk_hist = take(static_cast<size_t>(permute_num_chunks(M * k)) * E * sizeof(int32_t));
  p.offsets = take((E + 1) * sizeof(int32_t));
  p.sorted_pair = take(P * sizeof(int32_t));
  p.pos_of_pair = take(P * sizeof(int32_t));
  p.sorted_w = take(P * sizeof(float));
  p.a_codes = take(P * H);
  p.a_scales = take(P * (H / kBlock) * sizeof(float));
  p.h_codes = take(P * I);
  p.h_scales = take(P * (I / kBlock) * sizeof(float));
  p.contrib = take(P * H * sizeof(uint16_t));
  p.sync = take((2 * E + 2) * sizeof(int32_t));  // counters of the one-launch decode layer
  p.total = o;
  return p;
}

}  // namespace

extern "C" {

const char* qarl_status_string(int s) {
  switch (s) {
    case QARL_OK: return "ok";
    case QARL_ERR_INVALID_ARG: return "invalid argument";
    case QARL_ERR_UNSUPPORTED_SHAPE: return "unsupported shape";
    case QARL_ERR_MISALIGNED: return "misaligned pointer or stride";
    case QARL_ERR_WORKSPACE_TOO_SMALL: return "workspace too small";
    case QARL_ERR_UNSUPPORTED_DEVICE: return "unsupported device (needs compute capability 10.x)";
    case QARL_ERR_CUDA: return "CUDA error";
    case QARL_ERR_DEVICE_TIMEOUT: return "device-side wait timed out";
    case QARL_ERR_BAD_EXPERT_ID: return "expert id out of range or repeated within a token";
    default: return "unknown status";
  }
}

int qarl_create(qarl_ctx** out, int device) {
  if (!out) return QARL_ERR_INVALID_ARG;
  *out = nullptr;
  int count = 0;
  if (cudaGetDeviceCount(&count) != cudaSuccess || device < 0 || device >= count) {
    cudaGetLastError();
    return QARL_ERR_UNSUPPORTED_DEVICE;
  }
  cudaDeviceProp prop;
  if (cudaGetDeviceProperties(&prop, device) != cudaSuccess) return QARL_ERR_CUDA;
  if (prop.major != 10) return QARL_ERR_UNSUPPORTED_DEVICE;
  if (cudaSetDevice(device) != cudaSuccess) return QARL_ERR_CUDA;
  qarl_ctx* ctx = new (std::nothrow) qarl_ctx();
  if (!ctx) return QARL_ERR_CUDA;
  ctx->device = device;
  ctx->sm_count = prop.multiProcessorCount;
  ctx->launches = 0;
  ctx->err[0] = 0;
  void* fn = nullptr;
  cudaDriverEntryPointQueryResult qres;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess ||
      qres != cudaDriverEntryPointSuccess || !fn) {
    delete ctx;
    return QARL_ERR_CUDA;
  }
  ctx->encode = reinterpret_cast<EncodeTiledFn>(fn);
  if (cudaMalloc(&ctx->d_status, sizeof(int)) != cudaSuccess ||
      cudaMemset(ctx->d_status, 0, sizeof(int)) != cudaSuccess) {
    delete ctx;
    return QARL_ERR_CUDA;
  }
  *out = ctx;
  return QARL_OK;
}

void qarl_destroy(qarl_ctx* ctx) {
  if (!ctx) return;
  cudaSetDevice(ctx->device);
  cudaFree(ctx->d_status);
  delete ctx;
}

int qarl_poll_device_status(qarl_ctx* ctx, void* stream) {
  if (!ctx) return QARL_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  int h = 0;
  cudaError_t e = cudaMemcpyAsync(&h, ctx->d_status, sizeof(int), cudaMemcpyDeviceToHost, st);
  if (e == cudaSuccess) e = cudaMemsetAsync(ctx->d_status, 0, sizeof(int), st);
  if (e == cudaSuccess) e = cudaStreamSynchronize(st);
  if (e != cudaSuccess) return cuda_fail(ctx, e, "poll");
  return h;
}

const char* qarl_last_cuda_error(qarl_ctx* ctx) { return ctx ? ctx->err : ""; }
int64_t qarl_launch_count(qarl_ctx* ctx) { return ctx ? ctx->launches : 0; }

int qarl_profile_begin(qarl_ctx* ctx, int max_marks) {
  if (!ctx || max_marks < 2) return QARL_ERR_INVALID_ARG;
  if (!ctx->marks.empty()) return QARL_ERR_INVALID_ARG;  // already on
  ctx->marks.resize(static_cast<size_t>(max_marks));
  ctx->mark_stage.assign(static_cast<size_t>(max_marks), -1);
  ctx->marks_used = 0;
  for (size_t i = 0; i < ctx->marks.size(); ++i) {
    cudaError_t e = cudaEventCreate(&ctx->marks[i]);
    if (e != cudaSuccess) {
      for (size_t j = 0; j < i; ++j) cudaEventDestroy(ctx->marks[j]);
      ctx->marks.clear();
      return cuda_fail(ctx, e, "cudaEventCreate");
    }
  }
  return QARL_OK;
}

int qarl_profile_end(qarl_ctx* ctx, double* stage_ms, int64_t* stage_launches) {
  if (!ctx || !stage_ms || !stage_launches) return QARL_ERR_INVALID_ARG;
  cudaError_t e = cudaDeviceSynchronize();
  int rc = e == cudaSuccess ? QARL_OK : cuda_fail(ctx, e, "profile_end");
  for (size_t i = 1; rc == QARL_OK && i < ctx->marks_used; ++i) {
    const int st = ctx->mark_stage[i];
    if (st < 0 || st >= QARL_NUM_STAGES) continue;
    float ms = 0.f;
    if (cudaEventElapsedTime(&ms, ctx->marks[i - 1], ctx->marks[i]) == cudaSuccess) {
      stage_ms[st] += ms;
      stage_launches[st] += 1;
    }
  }
  for (cudaEvent_t ev : ctx->marks) cudaEventDestroy(ev);
  ctx->marks.clear();
  ctx->mark_stage.clear();
  ctx->marks_used = 0;
  return rc;
}

int qarl_quantize_weight(qarl_ctx* ctx, const void* w, int64_t E, int64_t N, int64_t K, uint8_t* codes,
                         float* scales, void* stream) {
  return qarl_quantize_weight_publish(ctx, w, E, N, K, codes, scales, nullptr, nullptr, stream);
}

int qarl_quantize_weight_publish(qarl_ctx* ctx, const void* w, int64_t E, int64_t N, int64_t K, uint8_t* codes,
                                 float* scales, uint8_t* pub_codes, float* pub_scales, void* stream) {
  NvtxRange nvtx_range("qarl_quantize_weight_publish");
  if (!ctx || E < 0 || N < 0 || K < 0) return QARL_ERR_INVALID_ARG;
  if ((pub_codes == nullptr) != (pub_scales == nullptr)) return QARL_ERR_INVALID_ARG;
  if (!aligned16(pub_codes) || (reinterpret_cast<uintptr_t>(pub_scales) & 3u)) return QARL_ERR_MISALIGNED;
  if (N % kBlock || K % kBlock) return QARL_ERR_UNSUPPORTED_SHAPE;
  if (E * (N / kBlock) * (K / kBlock) > 0x7FFFFFFFll) return QARL_ERR_UNSUPPORTED_SHAPE;
  if (E == 0 || N == 0 || K == 0) return QARL_OK;
  if (!w || !codes || !scales) return QARL_ERR_INVALID_ARG;
  if (!aligned16(w) || !aligned16(codes) || (reinterpret_cast<uintptr_t>(scales) & 3u)) return QARL_ERR_MISALIGNED;
  mark(ctx, static_cast<cudaStream_t>(stream), -1);
  cudaError_t e = launch_quantize_weight(make_launch(ctx, stream), static_cast<const uint16_t*>(w), E, N, K, codes,
                                         scales, pub_codes, pub_scales);
  mark(ctx, static_cast<cudaStream_t>(stream), QARL_STAGE_QUANT_WEIGHT);
  return e == cudaSuccess ? QARL_OK : cuda_fail(ctx, e, "quantize_weight");
}

int qarl_quantize_act(qarl_ctx* ctx, const void* x, int64_t M, int64_t K, int64_t ldx, uint8_t* codes,
                      float* scales, void* stream) {
  NvtxRange nvtx_range("qarl_quantize_act");
  if (!ctx || M < 0 || K < 0 || ldx < K) return QARL_ERR_INVALID_ARG;
  if (K % kBlock) return QARL_ERR_UNSUPPORTED_SHAPE;
  if (M * (K / kBlock) > (0x7FFFFFFFll << 5)) return QARL_ERR_UNSUPPORTED_SHAPE;
  if (M == 0 || K == 0) return QARL_OK;
  if (!x || !codes || !scales) return QARL_ERR_INVALID_ARG;
  if (!aligned16(x) || !aligned16(codes) || (ldx % 8) || (reinterpret_cast<uintptr_t>(scales) & 3u))
    return QARL_ERR_MISALIGNED;
  mark(ctx, static_cast<cudaStream_t>(stream), -1);
  cudaError_t e = launch_quantize_act(make_launch(ctx, stream), static_cast<const uint16_t*>(x), M, K, ldx, codes,
                                      scales, nullptr, 1);
  mark(ctx, static_cast<cudaStream_t>(stream), QARL_STAGE_QUANT_ACT);
  return e == cudaSuccess ? QARL_OK : cuda_fail(ctx, e, "quantize_act");
}

size_t qarl_linear_workspace_bytes(int64_t M, int64_t N, int64_t K) {
  (void)N;
  if (M <= 0 || K <= 0) return 0;
  return align_up(static_cast<size_t>(M) * K, 256) + align_up(static_cast<size_t>(M) * (K / kBlock) * sizeof(float), 256);
}

int qarl_linear_fwd_q(qarl_ctx* ctx, const uint8_t* xc, const float* xs, int64_t M, int64_t K, const uint8_t* wc,
                      const float* ws, int64_t N, void* y, float* y_f32, void* stream) {
  NvtxRange nvtx_range("qarl_linear_fwd_q");
  if (!ctx || M < 0 || K <= 0 || N <= 0) return QARL_ERR_INVALID_ARG;
  if (N % kBlock || K % kBlock || M > 0x7FFFFF00ll || N > 0x7FFFFF00ll) return QARL_ERR_UNSUPPORTED_SHAPE;
  if (M == 0) return QARL_OK;
  if (!xc || !xs || !wc || !ws || !y) return QARL_ERR_INVALID_ARG;
  if (!aligned16(xc) || !aligned16(wc) || !aligned16(y) || !aligned16(y_f32) ||
      (reinterpret_cast<uintptr_t>(xs) & 3u) || (reinterpret_cast<uintptr_t>(ws) & 3u))
    return QARL_ERR_MISALIGNED;
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
  a.out_f32 = y_f32;
  mark(ctx, static_cast<cudaStream_t>(stream), -1);
  const int rc = run_gemm(ctx, make_launch(ctx, stream), a);
  mark(ctx, static_cast<cudaStream_t>(stream), QARL_STAGE_LINEAR_GEMM);
  return rc;
}

int qarl_linear_fwd(qarl_ctx* ctx, const void* x, int64_t M, int64_t K, const uint8_t* wc, const float* ws,
                    int64_t N, void* y, float* y_f32, void* workspace, size_t workspace_bytes, void* stream) {
  NvtxRange nvtx_range("qarl_linear_fwd");
  if (!ctx || M < 0 || K <= 0 || N <= 0) return QARL_ERR_INVALID_ARG;
  if (N % kBlock || K % kBlock || M > 0x7FFFFF00ll || N > 0x7FFFFF00ll) return QARL_ERR_UNSUPPORTED_SHAPE;
  if (M == 0) return QARL_OK;
  if (!x || !wc || !ws || !y || !workspace) return QARL_ERR_INVALID_ARG;
  if (!aligned16(x) || (reinterpret_cast<uintptr_t>(workspace) & 255u)) return QARL_ERR_MISALIGNED;
  if (workspace_bytes < qarl_linear_workspace_bytes(M, N, K)) return QARL_ERR_WORKSPACE_TOO_SMALL;
  uint8_t* xc = static_cast<uint8_t*>(workspace);
  float* xs = reinterpret_cast<float*>(xc + align_up(static_cast<size_t>(M) * K, 256));
  mark(ctx, static_cast<cudaStream_t>(stream), -1);
  cudaError_t e = launch_quantize_act(make_launch(ctx, stream), static_cast<const uint16_t*>(x), M, K, K, xc, xs,
                                      nullptr, 1);
  mark(ctx, static_cast<cudaStream_t>(stream), QARL_STAGE_QUANT_ACT);
  if (e != cudaSuccess) return cuda_fail(ctx, e, "quantize_act");
  return qarl_linear_fwd_q(ctx, xc, xs, M, K, wc, ws, N, y, y_f32, stream);
}

size_t qarl_moe_workspace_bytes(int64_t M, int64_t H, int64_t I, int64_t E, int64_t k) {
  if (M <= 0 || H <= 0 || I <= 0 || E <= 0 || k <= 0) return 0;
  return plan_moe(M, H, I, E, k).total;
}

int qarl_moe_fwd(qarl_ctx* ctx, const void* x, const int32_t* ids, const float* wts, int64_t M, int64_t H,
                 int64_t I, int64_t E, int64_t k, const uint8_t* w13c, const float* w13s, const uint8_t* w2c,
                 const float* w2s, void* out, void* workspace, size_t workspace_bytes, const qarl_moe_debug* dbg,
                 void* stream) {
  NvtxRange nvtx_range("qarl_moe_fwd");
  if (!ctx || M < 0 || H <= 0 || I <= 0 || E < 1 || k < 1 || k > 32) return QARL_ERR_INVALID_ARG;
  if (H % kBlock || I % kBlock || E > 1024 || M * k >= 0x7FFFFF00ll || E * 2 * I > 0x7FFFFF00ll)
    return QARL_ERR_UNSUPPORTED_SHAPE;
  if (M == 0) return QARL_OK;
  if (!x || !ids || !wts || !w13c || !w13s || !w2c || !w2s || !out || !workspace) return QARL_ERR_INVALID_ARG;
  if (!aligned16(x) || !aligned16(w13c) || !aligned16(w2c) || !aligned16(out) ||
      (reinterpret_cast<uintptr_t>(workspace) & 255u))
    return QARL_ERR_MISALIGNED;
  const MoePlan pl = plan_moe(M, H, I, E, k);
  if (workspace_bytes < pl.total) return QARL_ERR_WORKSPACE_TOO_SMALL;
  uint8_t* ws = static_cast<uint8_t*>(workspace);
  const int64_t P = M * k;
  Launch L = make_launch(ctx, stream);
  cudaError_t e;

  PermuteBuffers pb;
  pb.chunk_hist = reinterpret_cast<int32_t*>(ws + pl.chunk_hist);
  pb.offsets = reinterpret_cast<int32_t*>(ws + pl.offsets);
  pb.sorted_pair = reinterpret_cast<int32_t*>(ws + pl.sorted_pair);
  pb.pos_of_pair = reinterpret_cast<int32_t*>(ws + pl.pos_of_pair);
  // Bad ids are skipped by the permutation and leave their entries of these arrays stale; every
  // consumer clamps the indices it reads from them, so no clearing pass is needed.
  uint8_t* a_codes = ws + pl.a_codes;
  float* a_scales = reinterpret_cast<float*>(ws + pl.a_scales);
  float* sorted_w = reinterpret_cast<float*>(ws + pl.sorted_w);
  int32_t* layer_sync = reinterpret_cast<int32_t*>(ws + pl.sync);
  const bool prep_small = moe_prep_small_applies(M, k, E);
  mark(ctx, L.stream, -1);
  if (prep_small) {
    // decode-sized: grouping + quantization + scatter in one launch (timed as the quantize_act stage)
    if ((e = launch_moe_prep_small(L, ids, M, k, E, pb, static_cast<const uint16_t*>(x), H, wts, a_codes, a_scales,
                                   sorted_w, layer_sync, static_cast<int>(2 * E + 2))) != cudaSuccess)
      return cuda_fail(ctx, e, "moe_prep");
    mark(ctx, L.stream, QARL_STAGE_QUANT_ACT);
  } else {
    if ((e = launch_permute(L, ids, M, k, E, pb)) != cudaSuccess) return cuda_fail(ctx, e, "permute");
    mark(ctx, L.stream, QARL_STAGE_PERMUTE);
    if ((e = launch_quantize_act(L, static_cast<const uint16_t*>(x), M, H, H, a_codes, a_scales, pb.pos_of_pair,
                                 static_cast<int>(k), wts, sorted_w)) != cudaSuccess)
      return cuda_fail(ctx, e, "quantize_act");
    mark(ctx, L.stream, QARL_STAGE_QUANT_ACT);
  }

  uint8_t* h_codes = ws + pl.h_codes;
  float* h_scales = reinterpret_cast<float*>(ws + pl.h_scales);
  GemmArgs g{};
  g.mode = kModeGateUp;
  g.a_codes = a_codes;
  g.a_scales = a_scales;
  g.rows_total = P;
  g.K = H;
  g.b_codes = w13c;
  g.b_scales = w13s;
  g.N = 2 * I;
  g.E = E;
  g.offsets = pb.offsets;
  g.out_bf16 = dbg ? static_cast<uint16_t*>(dbg->gate_up_bf16) : nullptr;
  g.h_codes = h_codes;
  g.h_scales = h_scales;
  g.h_bf16 = dbg ? static_cast<uint16_t*>(dbg->h_bf16) : nullptr;
  uint16_t* contrib = reinterpret_cast<uint16_t*>(ws + pl.contrib);
  GemmArgs d{};
  d.mode = kModeDown;
  d.a_codes = h_codes;
  d.a_scales = h_scales;
  d.rows_total = P;
  d.K = I;
  d.b_codes = w2c;
  d.b_scales = w2s;
  d.N = H;
  d.E = E;
  d.offsets = pb.offsets;
  d.out_bf16 = contrib;
  d.out_f32 = dbg ? dbg->down_f32 : nullptr;
  d.sorted_pair = nullptr;  // contributions stay in sorted order (dense row blocks); the k-sum finds them by position
  d.pair_weights = sorted_w;

  int rc;
  if (prep_small && L.gemm_path == 0 && moe_decode_layer_applies(g, d)) {
    // decode-sized: both projections and the k-sum in one launch (its counters were cleared by the
    // grouping kernel)
    CUresult cu = CUDA_SUCCESS;
    e = launch_moe_decode_layer(L, ctx->encode, g, d, ids, pb.pos_of_pair, M, k, static_cast<uint16_t*>(out),
                                layer_sync, &cu);
    if (cu != CUDA_SUCCESS) {
      snprintf(ctx->err, sizeof(ctx->err), "cuTensorMapEncodeTiled failed with CUresult %d", static_cast<int>(cu));
      return QARL_ERR_CUDA;
    }
    if (e != cudaSuccess) return cuda_fail(ctx, e, "moe decode layer launch");
    mark(ctx, L.stream, QARL_STAGE_MOE_DECODE_LAYER);
  } else {
    rc = run_gemm(ctx, L, g);
    if (rc != QARL_OK) return rc;
    mark(ctx, L.stream, QARL_STAGE_GATE_UP_GEMM);
    rc = run_gemm(ctx, L, d);
    if (rc != QARL_OK) return rc;
    mark(ctx, L.stream, QARL_STAGE_DOWN_GEMM);
    if ((e = launch_combine(L, contrib, ids, M, k, H, E, static_cast<uint16_t*>(out), pb.pos_of_pair)) != cudaSuccess)
      return cuda_fail(ctx, e, "combine");
    mark(ctx, L.stream, QARL_STAGE_COMBINE);
  }

  if (dbg) {
    if (dbg->expert_offsets &&
        (e = cudaMemcpyAsync(dbg->expert_offsets, pb.offsets, (E + 1) * sizeof(int32_t), cudaMemcpyDeviceToDevice,
                             L.stream)) != cudaSuccess)
      return cuda_fail(ctx, e, "copy offsets");
    if (dbg->sorted_pair && (e = cudaMemcpyAsync(dbg->sorted_pair, pb.sorted_pair, P * sizeof(int32_t),
                                                 cudaMemcpyDeviceToDevice, L.stream)) != cudaSuccess)
      return cuda_fail(ctx, e, "copy sorted_pair");
    if (dbg->h_codes && (e = cudaMemcpyAsync(dbg->h_codes, h_codes, static_cast<size_t>(P) * I,
                                             cudaMemcpyDeviceToDevice, L.stream)) != cudaSuccess)
      return cuda_fail(ctx, e, "copy h_codes");
    if (dbg->h_scales &&
        (e = cudaMemcpyAsync(dbg->h_scales, h_scales, static_cast<size_t>(P) * (I / kBlock) * sizeof(float),
                             cudaMemcpyDeviceToDevice, L.stream)) != cudaSuccess)
      return cuda_fail(ctx, e, "copy h_scales");
  }
  return QARL_OK;
}

int qarl_harness_rmsnorm(qarl_ctx* ctx, const void* x, int64_t M, int64_t H, float eps, void* out, void* stream) {
  if (!ctx || M < 0 || H <= 0) return QARL_ERR_INVALID_ARG;
  if (H % 8) return QARL_ERR_UNSUPPORTED_SHAPE;
  if (M == 0) return QARL_OK;
  if (!x || !out) return QARL_ERR_INVALID_ARG;
  if (!aligned16(x) || !aligned16(out)) return QARL_ERR_MISALIGNED;
  cudaError_t e = launch_rmsnorm(make_launch(ctx, stream), static_cast<const uint16_t*>(x), M, H, eps,
                                 static_cast<uint16_t*>(out));
  return e == cudaSuccess ? QARL_OK : cuda_fail(ctx, e, "rmsnorm");
}

int qarl_harness_set_wait_limit_ns(qarl_ctx* ctx, uint64_t limit_ns) {
  if (!ctx) return QARL_ERR_INVALID_ARG;
  if (limit_ns != 0) limit_ns = limit_ns < 1000 ? 1000 : (limit_ns > 2000000000ull ? 2000000000ull : limit_ns);
  ctx->wait_limit_ns = limit_ns;
  return QARL_OK;
}

int qarl_harness_set_gemm_path(qarl_ctx* ctx, int path) {
  if (!ctx || path < 0 || path > 2) return QARL_ERR_INVALID_ARG;
  ctx->gemm_path = path;
  return QARL_OK;
}

int qarl_harness_stop_producer_after(qarl_ctx* ctx, int64_t stages) {
  if (!ctx) return QARL_ERR_INVALID_ARG;
  ctx->stop_after_stages = stages < 0 ? -1 : static_cast<int>(stages > 0x7FFFFFFF ? 0x7FFFFFFF : stages);
  return QARL_OK;
}

int qarl_harness_fp8_mma_peak(qarl_ctx* ctx, int64_t kblocks_per_sm, double* flop_out, void* stream) {
  if (!ctx || kblocks_per_sm < 1 || kblocks_per_sm > 100000000ll) return QARL_ERR_INVALID_ARG;
  if (flop_out) *flop_out = 2.0 * 128 * 256 * 128 * static_cast<double>(kblocks_per_sm) * ctx->sm_count;
  cudaError_t e = launch_fp8_mma_peak(make_launch(ctx, stream), static_cast<int>(kblocks_per_sm));
  return e == cudaSuccess ? QARL_OK : cuda_fail(ctx, e, "fp8_mma_peak");
}

int qarl_harness_read_stream(qarl_ctx* ctx, const void* buf, size_t bytes, void* sink4, void* stream) {
  if (!ctx || !buf || !sink4) return QARL_ERR_INVALID_ARG;
  if (!aligned16(buf) || (reinterpret_cast<uintptr_t>(sink4) & 3u)) return QARL_ERR_MISALIGNED;
  cudaError_t e = launch_read_stream(make_launch(ctx, stream), buf, bytes, static_cast<uint32_t*>(sink4));
  return e == cudaSuccess ? QARL_OK : cuda_fail(ctx, e, "read_stream");
}

int qarl_harness_wait_selftest(qarl_ctx* ctx, uint64_t limit_ns, void* stream) {
  if (!ctx) return QARL_ERR_INVALID_ARG;
  if (limit_ns < 1000) limit_ns = 1000;
  if (limit_ns > 100000000ull) limit_ns = 100000000ull;
  cudaError_t e = launch_wait_selftest(make_launch(ctx, stream), limit_ns);
  return e == cudaSuccess ? QARL_OK : cuda_fail(ctx, e, "wait_selftest");
}

}  // extern "C"
