// Expert-parallel decomposition of the FP8 MoE layer: the three device stages between which the rows
// travel when the experts are split across GPUs (dispatch on the token's GPU, the two expert GEMMs on
// the expert's GPU, the k-sum back on the token's GPU).  Every stage is made of the same kernels as
// qarl_moe_fwd, and each row's arithmetic is unchanged, so by the row invariance (App. C) the result
// is bitwise that of the single-GPU layer.
#include "api_util.cuh"

namespace qarl {
namespace {

struct DispatchPlan {
  size_t chunk_hist, sorted_pair, total;
};
DispatchPlan plan_dispatch(int64_t M, int64_t E, int64_t k) {
  DispatchPlan p{};
  size_t o = 0;
  auto take = [&](size_t bytes) {
    const size_t at = o;
    o += (bytes + 255) & ~static_cast<size_t>(255);
    return at;
  };
  p.chunk_hist = take(static_cast<size_t>(permute_num_chunks(M * k)) * E * sizeof(int32_t));
  p.sorted_pair = take(static_cast<size_t>(M * k) * sizeof(int32_t));
  p.total = o;
  return p;
}

struct ExpertsPlan {
  size_t h_codes, h_scales, total;
};
ExpertsPlan plan_experts(int64_t R, int64_t I) {
  ExpertsPlan p{};
  size_t o = 0;
  auto take = [&](size_t bytes) {
    const size_t at = o;
    o += (bytes + 255) & ~static_cast<size_t>(255);
    return at;
  };
  p.h_codes = take(static_cast<size_t>(R) * I);
  p.h_scales = take(static_cast<size_t>(R) * (I / kBlock) * sizeof(float));
  p.total = o;
  return p;
}

}  // namespace
}  // namespace qarl

using namespace qarl;

extern "C" {

size_t qarl_moe_dispatch_workspace_bytes(int64_t M, int64_t E, int64_t k) {
  if (M <= 0 || E <= 0 || k <= 0) return 0;
  return plan_dispatch(M, E, k).total;
}

int qarl_moe_dispatch(qarl_ctx* ctx, const void* x, const int32_t* ids, const float* wts, int64_t M, int64_t H,
                      int64_t E, int64_t k, uint8_t* codes_sorted, float* scales_sorted, float* weights_sorted,
                      int32_t* offsets, int32_t* pos_of_pair, void* workspace, size_t workspace_bytes, void* stream) {
  NvtxRange nvtx_range("qarl_moe_dispatch");
  if (!ctx || M < 0 || H <= 0 || E < 1 || k < 1 || k > 32) return QARL_ERR_INVALID_ARG;
  if (H % kBlock || E > 1024 || M * k >= 0x7FFFFF00ll) return QARL_ERR_UNSUPPORTED_SHAPE;
  if (!offsets) return QARL_ERR_INVALID_ARG;
  Launch L = make_launch(ctx, stream);
  cudaError_t e;
  if (M == 0) {  // no pairs: every group is empty
    if ((e = cudaMemsetAsync(offsets, 0, (E + 1) * sizeof(int32_t), L.stream)) != cudaSuccess)
      return cuda_fail(ctx, e, "dispatch offsets");
    return QARL_OK;
  }
  if (!x || !ids || !wts || !codes_sorted || !scales_sorted || !weights_sorted || !pos_of_pair || !workspace)
    return QARL_ERR_INVALID_ARG;
  if (!aligned16(x) || !aligned16(codes_sorted) || (reinterpret_cast<uintptr_t>(workspace) & 255u))
    return QARL_ERR_MISALIGNED;
  const DispatchPlan pl = plan_dispatch(M, E, k);
  if (workspace_bytes < pl.total) return QARL_ERR_WORKSPACE_TOO_SMALL;
  uint8_t* ws = static_cast<uint8_t*>(workspace);
  PermuteBuffers pb;
  pb.chunk_hist = reinterpret_cast<int32_t*>(ws + pl.chunk_hist);
  pb.offsets = offsets;
  pb.sorted_pair = reinterpret_cast<int32_t*>(ws + pl.sorted_pair);
  pb.pos_of_pair = pos_of_pair;
  mark(ctx, L.stream, -1);
  if ((e = launch_permute(L, ids, M, k, E, pb)) != cudaSuccess) return cuda_fail(ctx, e, "permute");
  mark(ctx, L.stream, QARL_STAGE_PERMUTE);
  if ((e = launch_quantize_act(L, static_cast<const uint16_t*>(x), M, H, H, codes_sorted, scales_sorted, pos_of_pair,
                               static_cast<int>(k), wts, weights_sorted)) != cudaSuccess)
    return cuda_fail(ctx, e, "quantize_act");
  mark(ctx, L.stream, QARL_STAGE_QUANT_ACT);
  return QARL_OK;
}

size_t qarl_moe_experts_workspace_bytes(int64_t R, int64_t I) {
  if (R <= 0 || I <= 0) return 0;
  return plan_experts(R, I).total;
}

int qarl_moe_experts_fwd(qarl_ctx* ctx, const uint8_t* codes, const float* scales, const float* row_weights,
                         const int32_t* offsets, int64_t R, int64_t H, int64_t I, int64_t E_local,
                         const uint8_t* w13c, const float* w13s, const uint8_t* w2c, const float* w2s, void* contrib,
                         void* workspace, size_t workspace_bytes, void* stream) {
  NvtxRange nvtx_range("qarl_moe_experts_fwd");
  if (!ctx || R < 0 || H <= 0 || I <= 0 || E_local < 1) return QARL_ERR_INVALID_ARG;
  if (H % kBlock || I % kBlock || E_local > 1024 || R >= 0x7FFFFF00ll || E_local * 2 * I > 0x7FFFFF00ll)
    return QARL_ERR_UNSUPPORTED_SHAPE;
  if (R == 0) return QARL_OK;
  if (!codes || !scales || !row_weights || !offsets || !w13c || !w13s || !w2c || !w2s || !contrib || !workspace)
    return QARL_ERR_INVALID_ARG;
  if (!aligned16(codes) || !aligned16(w13c) || !aligned16(w2c) || !aligned16(contrib) ||
      (reinterpret_cast<uintptr_t>(workspace) & 255u))
    return QARL_ERR_MISALIGNED;
  const ExpertsPlan pl = plan_experts(R, I);
  if (workspace_bytes < pl.total) return QARL_ERR_WORKSPACE_TOO_SMALL;
  uint8_t* ws = static_cast<uint8_t*>(workspace);
  Launch L = make_launch(ctx, stream);
  uint8_t* h_codes = ws + pl.h_codes;
  float* h_scales = reinterpret_cast<float*>(ws + pl.h_scales);
  mark(ctx, L.stream, -1);
  GemmArgs g{};
  g.mode = kModeGateUp;
  g.a_codes = codes;
  g.a_scales = scales;
  g.rows_total = R;
  g.K = H;
  g.b_codes = w13c;
  g.b_scales = w13s;
  g.N = 2 * I;
  g.E = E_local;
  g.offsets = offsets;
  g.h_codes = h_codes;
  g.h_scales = h_scales;
  int rc = run_gemm(ctx, L, g);
  if (rc != QARL_OK) return rc;
  mark(ctx, L.stream, QARL_STAGE_GATE_UP_GEMM);
  GemmArgs d{};
  d.mode = kModeDown;
  d.a_codes = h_codes;
  d.a_scales = h_scales;
  d.rows_total = R;
  d.K = I;
  d.b_codes = w2c;
  d.b_scales = w2s;
  d.N = H;
  d.E = E_local;
  d.offsets = offsets;
  d.out_bf16 = static_cast<uint16_t*>(contrib);
  d.sorted_pair = nullptr;  // contributions stay in the order the rows came in
  d.pair_weights = row_weights;
  rc = run_gemm(ctx, L, d);
  if (rc != QARL_OK) return rc;
  mark(ctx, L.stream, QARL_STAGE_DOWN_GEMM);
  return QARL_OK;
}

int qarl_moe_combine_sorted(qarl_ctx* ctx, const void* contrib_sorted, const int32_t* ids, const int32_t* pos_of_pair,
                            int64_t M, int64_t H, int64_t E, int64_t k, void* out, void* stream) {
  NvtxRange nvtx_range("qarl_moe_combine_sorted");
  if (!ctx || M < 0 || H <= 0 || E < 1 || k < 1 || k > 32) return QARL_ERR_INVALID_ARG;
  if (H % 8 || M * k >= 0x7FFFFF00ll) return QARL_ERR_UNSUPPORTED_SHAPE;
  if (M == 0) return QARL_OK;
  if (!contrib_sorted || !ids || !pos_of_pair || !out) return QARL_ERR_INVALID_ARG;
  if (!aligned16(contrib_sorted) || !aligned16(out)) return QARL_ERR_MISALIGNED;
  Launch L = make_launch(ctx, stream);
  mark(ctx, L.stream, -1);
  cudaError_t e = launch_combine(L, static_cast<const uint16_t*>(contrib_sorted), ids, M, k, H, E,
                                 static_cast<uint16_t*>(out), pos_of_pair);
  mark(ctx, L.stream, QARL_STAGE_COMBINE);
  return e == cudaSuccess ? QARL_OK : cuda_fail(ctx, e, "combine");
}

}  // extern "C"
