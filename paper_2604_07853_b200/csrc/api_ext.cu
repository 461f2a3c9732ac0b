// C ABI entry points beyond the FP8 forward: the W4A16 path (4-bit group-quantized weights, bf16
// activations), the full-precision backward (dense, per expert, whole layer), the TBPO loss and the
// router: argument checks, workspace planning, kernel sequencing.  No device memory is allocated here.
#include "api_util.cuh"

namespace {

using namespace qarl;

int run_gemm_w4(qarl_ctx* ctx, const Launch& L, const GemmW4Args& a) {
  CUresult cu = CUDA_SUCCESS;
  cudaError_t e = launch_gemm_w4a16(L, ctx->encode, a, &cu);
  if (cu != CUDA_SUCCESS) {
    snprintf(ctx->err, sizeof(ctx->err), "cuTensorMapEncodeTiled failed with CUresult %d", static_cast<int>(cu));
    return QARL_ERR_CUDA;
  }
  if (e != cudaSuccess) return cuda_fail(ctx, e, "w4a16 gemm launch");
  return QARL_OK;
}

// Workspace carve-up of qarl_moe_bwd.
struct MoeBwdPlan {
  size_t chunk_hist, offsets, sorted_pair, pos_of_pair, sorted_w, x_sorted, dy, dh, dgu, dxs, total;
};
MoeBwdPlan plan_moe_bwd(int64_t M, int64_t H, int64_t I, int64_t E, int64_t k) {
  const size_t P = static_cast<size_t>(M * k);
  MoeBwdPlan p{};
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
  p.x_sorted = take(P * H * sizeof(uint16_t));
  p.dy = take(P * H * sizeof(uint16_t));
  p.dh = take(P * I * sizeof(uint16_t));
  p.dgu = take(P * 2 * I * sizeof(uint16_t));
  p.dxs = take(P * H * sizeof(uint16_t));
  p.total = o;
  return p;
}

// Workspace carve-up of qarl_moe_fwd_w4a16; every slice starts on a 256-byte boundary.
struct MoeW4Plan {
  size_t chunk_hist, offsets, sorted_pair, pos_of_pair, sorted_w, x_sorted, h, contrib, total;
};
MoeW4Plan plan_moe_w4(int64_t M, int64_t H, int64_t I, int64_t E, int64_t k) {
  const size_t P = static_cast<size_t>(M * k);
  MoeW4Plan p{};
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
  p.x_sorted = take(P * H * sizeof(uint16_t));
  p.h = take(P * I * sizeof(uint16_t));
  p.contrib = take(P * H * sizeof(uint16_t));
  p.total = o;
  return p;
}

int quantize_w4(qarl_ctx* ctx, int fmt, const void* w, int64_t E, int64_t N, int64_t K, uint8_t* packed,
                void* scales, uint8_t* zeros, uint8_t* pub_packed, void* pub_scales, uint8_t* pub_zeros,
                void* stream) {
  if (!ctx || E < 0 || N < 0 || K < 0) return QARL_ERR_INVALID_ARG;
  const bool int4 = fmt == kFmtInt4;
  const int npub = (pub_packed != nullptr) + (pub_scales != nullptr) + (pub_zeros != nullptr);
  if (npub != 0 && npub != (int4 ? 3 : 2)) return QARL_ERR_INVALID_ARG;
  if (!aligned16(pub_packed) || (reinterpret_cast<uintptr_t>(pub_scales) & 1u)) return QARL_ERR_MISALIGNED;
  if (K % kBlock || N % kBlock) return QARL_ERR_UNSUPPORTED_SHAPE;
  if (E * N * (K / kBlock) >= 0x10000000ll || E * N >= 0x7FFFFFFFll) return QARL_ERR_UNSUPPORTED_SHAPE;  // 32-bit group index x 8 threads
  if (E == 0 || N == 0 || K == 0) return QARL_OK;
  if (!w || !packed || !scales || (int4 && !zeros)) return QARL_ERR_INVALID_ARG;
  if (!aligned16(w) || !aligned16(packed) || (reinterpret_cast<uintptr_t>(scales) & 1u)) return QARL_ERR_MISALIGNED;
  mark(ctx, static_cast<cudaStream_t>(stream), -1);
  cudaError_t e = launch_quantize_weight_w4(make_launch(ctx, stream), fmt, static_cast<const uint16_t*>(w), E, N, K, packed,
                                            static_cast<uint16_t*>(scales), zeros, pub_packed,
                                            static_cast<uint16_t*>(pub_scales), pub_zeros);
  mark(ctx, static_cast<cudaStream_t>(stream), QARL_STAGE_QUANT_WEIGHT);
  return e == cudaSuccess ? QARL_OK : cuda_fail(ctx, e, "quantize_weight_w4");
}

int linear_w4(qarl_ctx* ctx, int fmt, const void* x, int64_t M, int64_t K, const uint8_t* wp, const void* ws,
              const uint8_t* wz, int64_t N, void* y, float* y_f32, void* stream) {
  if (!ctx || M < 0 || K <= 0 || N <= 0) return QARL_ERR_INVALID_ARG;
  if (N % kBlock || K % kBlock || M > 0x7FFFFF00ll || N > 0x7FFFFF00ll) return QARL_ERR_UNSUPPORTED_SHAPE;
  if (M == 0) return QARL_OK;
  if (!x || !wp || !ws || (fmt == kFmtInt4 && !wz) || !y) return QARL_ERR_INVALID_ARG;
  if (!aligned16(x) || !aligned16(wp) || !aligned16(y) || !aligned16(y_f32) ||
      (reinterpret_cast<uintptr_t>(ws) & 1u))
    return QARL_ERR_MISALIGNED;
  GemmW4Args a{};
  a.mode = kModeLinear;
  a.fmt = fmt;
  a.a_bf16 = static_cast<const uint16_t*>(x);
  a.rows_total = M;
  a.K = K;
  a.b_packed = wp;
  a.b_scales = static_cast<const uint16_t*>(ws);
  a.b_zeros = wz;
  a.N = N;
  a.E = 1;
  a.out_bf16 = static_cast<uint16_t*>(y);
  a.out_f32 = y_f32;
  mark(ctx, static_cast<cudaStream_t>(stream), -1);
  const int rc = run_gemm_w4(ctx, make_launch(ctx, stream), a);
  mark(ctx, static_cast<cudaStream_t>(stream), QARL_STAGE_LINEAR_GEMM);
  return rc;
}

int moe_w4(qarl_ctx* ctx, int fmt, const void* x, const int32_t* ids, const float* wts, int64_t M, int64_t H,
           int64_t I, int64_t E, int64_t k, const uint8_t* w13p, const void* w13s, const uint8_t* w13z,
           const uint8_t* w2p, const void* w2s, const uint8_t* w2z, void* out, void* workspace,
           size_t workspace_bytes, const qarl_moe_debug* dbg, void* stream) {
  if (!ctx || M < 0 || H <= 0 || I <= 0 || E < 1 || k < 1 || k > 32) return QARL_ERR_INVALID_ARG;
  // the down tile spans 256 adjacent weight rows of one expert
  if (H % 256 || I % kBlock || E > 1024 || M * k >= 0x7FFFFF00ll || E * 2 * I > 0x7FFFFF00ll)
    return QARL_ERR_UNSUPPORTED_SHAPE;
  if (M == 0) return QARL_OK;
  if (!x || !ids || !wts || !w13p || !w13s || !w2p || !w2s || !out || !workspace) return QARL_ERR_INVALID_ARG;
  if (fmt == kFmtInt4 && (!w13z || !w2z)) return QARL_ERR_INVALID_ARG;
  if (!aligned16(x) || !aligned16(w13p) || !aligned16(w2p) || !aligned16(out) ||
      (reinterpret_cast<uintptr_t>(w13s) & 1u) || (reinterpret_cast<uintptr_t>(w2s) & 1u) ||
      (reinterpret_cast<uintptr_t>(workspace) & 255u))
    return QARL_ERR_MISALIGNED;
  const MoeW4Plan pl = plan_moe_w4(M, H, I, E, k);
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
  mark(ctx, L.stream, -1);
  if ((e = launch_permute(L, ids, M, k, E, pb)) != cudaSuccess) return cuda_fail(ctx, e, "permute");
  mark(ctx, L.stream, QARL_STAGE_PERMUTE);

  uint16_t* x_sorted = reinterpret_cast<uint16_t*>(ws + pl.x_sorted);
  float* sorted_w = reinterpret_cast<float*>(ws + pl.sorted_w);
  if ((e = launch_scatter_rows(L, static_cast<const uint16_t*>(x), M, H, x_sorted, pb.pos_of_pair,
                               static_cast<int>(k), wts, sorted_w)) != cudaSuccess)
    return cuda_fail(ctx, e, "scatter_rows");
  mark(ctx, L.stream, QARL_STAGE_QUANT_ACT);

  uint16_t* h = reinterpret_cast<uint16_t*>(ws + pl.h);
  GemmW4Args g{};
  g.mode = kModeGateUp;
  g.fmt = fmt;
  g.a_bf16 = x_sorted;
  g.rows_total = P;
  g.K = H;
  g.b_packed = w13p;
  g.b_scales = static_cast<const uint16_t*>(w13s);
  g.b_zeros = w13z;
  g.N = 2 * I;
  g.E = E;
  g.offsets = pb.offsets;
  g.out_bf16 = dbg ? static_cast<uint16_t*>(dbg->gate_up_bf16) : nullptr;
  g.h_bf16 = h;
  int rc = run_gemm_w4(ctx, L, g);
  if (rc != QARL_OK) return rc;
  mark(ctx, L.stream, QARL_STAGE_GATE_UP_GEMM);

  uint16_t* contrib = reinterpret_cast<uint16_t*>(ws + pl.contrib);
  GemmW4Args d{};
  d.mode = kModeDown;
  d.fmt = fmt;
  d.a_bf16 = h;
  d.rows_total = P;
  d.K = I;
  d.b_packed = w2p;
  d.b_scales = static_cast<const uint16_t*>(w2s);
  d.b_zeros = w2z;
  d.N = H;
  d.E = E;
  d.offsets = pb.offsets;
  d.out_bf16 = contrib;
  d.out_f32 = dbg ? dbg->down_f32 : nullptr;
  d.sorted_pair = nullptr;  // contributions stay in sorted order (dense row blocks); the k-sum finds them by position
  d.pair_weights = sorted_w;
  rc = run_gemm_w4(ctx, L, d);
  if (rc != QARL_OK) return rc;
  mark(ctx, L.stream, QARL_STAGE_DOWN_GEMM);

  if ((e = launch_combine(L, contrib, ids, M, k, H, E, static_cast<uint16_t*>(out), pb.pos_of_pair)) != cudaSuccess)
    return cuda_fail(ctx, e, "combine");
  mark(ctx, L.stream, QARL_STAGE_COMBINE);

  if (dbg) {
    if (dbg->expert_offsets &&
        (e = cudaMemcpyAsync(dbg->expert_offsets, pb.offsets, (E + 1) * sizeof(int32_t), cudaMemcpyDeviceToDevice,
                             L.stream)) != cudaSuccess)
      return cuda_fail(ctx, e, "copy offsets");
    if (dbg->sorted_pair && (e = cudaMemcpyAsync(dbg->sorted_pair, pb.sorted_pair, P * sizeof(int32_t),
                                                 cudaMemcpyDeviceToDevice, L.stream)) != cudaSuccess)
      return cuda_fail(ctx, e, "copy sorted_pair");
    if (dbg->h_bf16 && (e = cudaMemcpyAsync(dbg->h_bf16, h, static_cast<size_t>(P) * I * sizeof(uint16_t),
                                            cudaMemcpyDeviceToDevice, L.stream)) != cudaSuccess)
      return cuda_fail(ctx, e, "copy h");
  }
  return QARL_OK;
}

}  // namespace

extern "C" {

int qarl_quantize_weight_w4(qarl_ctx* ctx, const void* w, int64_t E, int64_t N, int64_t K, uint8_t* packed,
                            void* scales, uint8_t* zeros, void* stream) {
  return quantize_w4(ctx, kFmtInt4, w, E, N, K, packed, scales, zeros, nullptr, nullptr, nullptr, stream);
}

int qarl_quantize_weight_w4_publish(qarl_ctx* ctx, const void* w, int64_t E, int64_t N, int64_t K, uint8_t* packed,
                                    void* scales, uint8_t* zeros, uint8_t* pub_packed, void* pub_scales,
                                    uint8_t* pub_zeros, void* stream) {
  return quantize_w4(ctx, kFmtInt4, w, E, N, K, packed, scales, zeros, pub_packed, pub_scales, pub_zeros, stream);
}

int qarl_quantize_weight_fp4(qarl_ctx* ctx, const void* w, int64_t E, int64_t N, int64_t K, uint8_t* packed,
                             void* scales, uint8_t* pub_packed, void* pub_scales, void* stream) {
  return quantize_w4(ctx, kFmtE2m1, w, E, N, K, packed, scales, nullptr, pub_packed, pub_scales, nullptr, stream);
}

int qarl_linear_fwd_w4a16(qarl_ctx* ctx, const void* x, int64_t M, int64_t K, const uint8_t* wp, const void* ws,
                          const uint8_t* wz, int64_t N, void* y, float* y_f32, void* stream) {
  return linear_w4(ctx, kFmtInt4, x, M, K, wp, ws, wz, N, y, y_f32, stream);
}

int qarl_linear_fwd_fp4a16(qarl_ctx* ctx, const void* x, int64_t M, int64_t K, const uint8_t* wp, const void* ws,
                           int64_t N, void* y, float* y_f32, void* stream) {
  return linear_w4(ctx, kFmtE2m1, x, M, K, wp, ws, nullptr, N, y, y_f32, stream);
}

int qarl_moe_fwd_w4a16(qarl_ctx* ctx, const void* x, const int32_t* ids, const float* wts, int64_t M, int64_t H,
                       int64_t I, int64_t E, int64_t k, const uint8_t* w13p, const void* w13s, const uint8_t* w13z,
                       const uint8_t* w2p, const void* w2s, const uint8_t* w2z, void* out, void* workspace,
                       size_t workspace_bytes, const qarl_moe_debug* dbg, void* stream) {
  NvtxRange nvtx_range("qarl_moe_fwd_w4a16");
  return moe_w4(ctx, kFmtInt4, x, ids, wts, M, H, I, E, k, w13p, w13s, w13z, w2p, w2s, w2z, out, workspace,
                workspace_bytes, dbg, stream);
}

int qarl_moe_fwd_fp4a16(qarl_ctx* ctx, const void* x, const int32_t* ids, const float* wts, int64_t M, int64_t H,
                        int64_t I, int64_t E, int64_t k, const uint8_t* w13p, const void* w13s, const uint8_t* w2p,
                        const void* w2s, void* out, void* workspace, size_t workspace_bytes,
                        const qarl_moe_debug* dbg, void* stream) {
  NvtxRange nvtx_range("qarl_moe_fwd_fp4a16");
  return moe_w4(ctx, kFmtE2m1, x, ids, wts, M, H, I, E, k, w13p, w13s, nullptr, w2p, w2s, nullptr, out, workspace,
                workspace_bytes, dbg, stream);
}

size_t qarl_moe_w4a16_workspace_bytes(int64_t M, int64_t H, int64_t I, int64_t E, int64_t k) {
  if (M <= 0 || H <= 0 || I <= 0 || E <= 0 || k <= 0) return 0;
  return plan_moe_w4(M, H, I, E, k).total;
}

int qarl_linear_bwd(qarl_ctx* ctx, const void* dy, const void* x, const void* w, int64_t M, int64_t N, int64_t K,
                    void* dx, float* dx_f32, float* dw_f32, void* stream) {
  NvtxRange nvtx_range("qarl_linear_bwd");
  if (!ctx || M < 0 || N <= 0 || K <= 0) return QARL_ERR_INVALID_ARG;
  if (N % 8 || K % 8 || M > 0x7FFFFF00ll || N > 0x7FFFFF00ll || K > 0x7FFFFF00ll) return QARL_ERR_UNSUPPORTED_SHAPE;
  if (M == 0) return QARL_OK;
  if (!dy || !x || !w) return QARL_ERR_INVALID_ARG;
  if (!aligned16(dy) || !aligned16(x) || !aligned16(w) || !aligned16(dx) || !aligned16(dx_f32) || !aligned16(dw_f32))
    return QARL_ERR_MISALIGNED;
  Launch L = make_launch(ctx, stream);
  CUresult cu = CUDA_SUCCESS;
  auto run = [&](const GemmBf16Args& a, const char* what) {
    cudaError_t e = launch_gemm_bf16(L, ctx->encode, a, &cu);
    if (cu != CUDA_SUCCESS) {
      snprintf(ctx->err, sizeof(ctx->err), "cuTensorMapEncodeTiled failed with CUresult %d", static_cast<int>(cu));
      return static_cast<int>(QARL_ERR_CUDA);
    }
    return e == cudaSuccess ? static_cast<int>(QARL_OK) : cuda_fail(ctx, e, what);
  };
  mark(ctx, L.stream, -1);
  if (dx || dx_f32) {
    GemmBf16Args a{};
    a.a = static_cast<const uint16_t*>(dy);  // A(m, n) = dY[m, n]: the contraction index n is contiguous
    a.a_mn_major = false;
    a.b = static_cast<const uint16_t*>(w);   // B(k, n) = W[n, k]: stored [n][k], the output index k is contiguous
    a.b_mn_major = true;
    a.Mo = M;
    a.No = K;
    a.Kc = N;
    a.c_bf16 = static_cast<uint16_t*>(dx);
    a.c_f32 = dx_f32;
    const int rc = run(a, "linear_bwd dX");
    if (rc != QARL_OK) return rc;
    mark(ctx, L.stream, QARL_STAGE_BWD_DX);
  }
  if (dw_f32) {
    GemmBf16Args a{};
    a.a = static_cast<const uint16_t*>(dy);  // A(n, m) = dY[m, n]: stored [m][n], the output index n is contiguous
    a.a_mn_major = true;
    a.b = static_cast<const uint16_t*>(x);   // B(k, m) = X[m, k]
    a.b_mn_major = true;
    a.Mo = N;
    a.No = K;
    a.Kc = M;
    a.c_f32 = dw_f32;
    const int rc = run(a, "linear_bwd dW");
    if (rc != QARL_OK) return rc;
    mark(ctx, L.stream, QARL_STAGE_BWD_DW);
  }
  return QARL_OK;
}

int qarl_grouped_linear_bwd(qarl_ctx* ctx, const void* dy, const void* x, const void* w, const int32_t* offsets,
                            int64_t P, int64_t N, int64_t K, int64_t E, void* dx, float* dx_f32, float* dw_f32,
                            void* stream) {
  NvtxRange nvtx_range("qarl_grouped_linear_bwd");
  if (!ctx || P < 0 || N <= 0 || K <= 0 || E < 1) return QARL_ERR_INVALID_ARG;
  if (N % 64 || K % 8 || E > 1024 || P > 0x7FFFFF00ll || E * N > 0x7FFFFF00ll || E * K > 0x7FFFFF00ll)
    return QARL_ERR_UNSUPPORTED_SHAPE;
  if (!w || !offsets || (P > 0 && (!dy || !x))) return QARL_ERR_INVALID_ARG;
  if (!aligned16(dy) || !aligned16(x) || !aligned16(w) || !aligned16(dx) || !aligned16(dx_f32) || !aligned16(dw_f32))
    return QARL_ERR_MISALIGNED;
  Launch L = make_launch(ctx, stream);
  CUresult cu = CUDA_SUCCESS;
  auto run = [&](const GemmBf16Args& a, const char* what) {
    cudaError_t e = launch_gemm_bf16(L, ctx->encode, a, &cu);
    if (cu != CUDA_SUCCESS) {
      snprintf(ctx->err, sizeof(ctx->err), "cuTensorMapEncodeTiled failed with CUresult %d", static_cast<int>(cu));
      return static_cast<int>(QARL_ERR_CUDA);
    }
    return e == cudaSuccess ? static_cast<int>(QARL_OK) : cuda_fail(ctx, e, what);
  };
  mark(ctx, L.stream, -1);
  if ((dx || dx_f32) && P > 0) {
    GemmBf16Args a{};
    a.group = 1;
    a.a = static_cast<const uint16_t*>(dy);  // A(p, n) = dY[p, n]
    a.b = static_cast<const uint16_t*>(w);   // B_e(k, n) = W_e[n, k]: stored [n][k], MN-major
    a.b_mn_major = true;
    a.Mo = P;
    a.No = K;
    a.Kc = N;
    a.E = E;
    a.offsets = offsets;
    a.c_bf16 = static_cast<uint16_t*>(dx);
    a.c_f32 = dx_f32;
    const int rc = run(a, "grouped_linear_bwd dX");
    if (rc != QARL_OK) return rc;
    mark(ctx, L.stream, QARL_STAGE_BWD_DX);
  }
  if (dw_f32) {
    if (P == 0) {  // no rows at all: every dW_e is zero
      cudaError_t e = cudaMemsetAsync(dw_f32, 0, static_cast<size_t>(E) * N * K * sizeof(float), L.stream);
      if (e != cudaSuccess) return cuda_fail(ctx, e, "grouped_linear_bwd dW");
      return QARL_OK;
    }
    GemmBf16Args a{};
    a.group = 2;
    a.a = static_cast<const uint16_t*>(dy);  // A(n, p) = dY[p, n]
    a.a_mn_major = true;
    a.b = static_cast<const uint16_t*>(x);   // B(k, p) = X[p, k]
    a.b_mn_major = true;
    a.Mo = N;
    a.No = K;
    a.E = E;
    a.offsets = offsets;
    a.rows_total = P;
    a.c_f32 = dw_f32;
    const int rc = run(a, "grouped_linear_bwd dW");
    if (rc != QARL_OK) return rc;
    mark(ctx, L.stream, QARL_STAGE_BWD_DW);
  }
  return QARL_OK;
}

size_t qarl_moe_bwd_workspace_bytes(int64_t M, int64_t H, int64_t I, int64_t E, int64_t k) {
  if (M <= 0 || H <= 0 || I <= 0 || E <= 0 || k <= 0) return 0;
  return plan_moe_bwd(M, H, I, E, k).total;
}

int qarl_moe_bwd(qarl_ctx* ctx, const void* x, const int32_t* ids, const float* wts, int64_t M, int64_t H, int64_t I,
                 int64_t E, int64_t k, const void* w13, const void* w2, const void* gate_up, const void* h,
                 const void* dout, const float* down_f32, void* dx, float* dw13, float* dw2, float* dwts,
                 void* workspace, size_t workspace_bytes, void* stream) {
  NvtxRange nvtx_range("qarl_moe_bwd");
  if (!ctx || M < 0 || H <= 0 || I <= 0 || E < 1 || k < 1 || k > 32) return QARL_ERR_INVALID_ARG;
  if (H % 64 || I % 32 || E > 1024 || M * k >= 0x7FFFFF00ll || E * 2 * I > 0x7FFFFF00ll || E * H > 0x7FFFFF00ll)
    return QARL_ERR_UNSUPPORTED_SHAPE;
  if (!w13 || !w2 || !dw13 || !dw2) return QARL_ERR_INVALID_ARG;
  if (!aligned16(w13) || !aligned16(w2) || !aligned16(dw13) || !aligned16(dw2)) return QARL_ERR_MISALIGNED;
  Launch L = make_launch(ctx, stream);
  cudaError_t e;
  if (M == 0) {  // no tokens: the weight gradients are zero
    if ((e = cudaMemsetAsync(dw13, 0, static_cast<size_t>(E) * 2 * I * H * sizeof(float), L.stream)) != cudaSuccess ||
        (e = cudaMemsetAsync(dw2, 0, static_cast<size_t>(E) * H * I * sizeof(float), L.stream)) != cudaSuccess)
      return cuda_fail(ctx, e, "moe_bwd");
    return QARL_OK;
  }
  if (!x || !ids || !wts || !gate_up || !h || !dout || !dx || !workspace) return QARL_ERR_INVALID_ARG;
  if (!aligned16(x) || !aligned16(gate_up) || !aligned16(h) || !aligned16(dout) || !aligned16(dx) ||
      !aligned16(down_f32) || (reinterpret_cast<uintptr_t>(workspace) & 255u))
    return QARL_ERR_MISALIGNED;
  const MoeBwdPlan pl = plan_moe_bwd(M, H, I, E, k);
  if (workspace_bytes < pl.total) return QARL_ERR_WORKSPACE_TOO_SMALL;
  uint8_t* ws = static_cast<uint8_t*>(workspace);
  const int64_t P = M * k;
  PermuteBuffers pb;
  pb.chunk_hist = reinterpret_cast<int32_t*>(ws + pl.chunk_hist);
  pb.offsets = reinterpret_cast<int32_t*>(ws + pl.offsets);
  pb.sorted_pair = reinterpret_cast<int32_t*>(ws + pl.sorted_pair);
  pb.pos_of_pair = reinterpret_cast<int32_t*>(ws + pl.pos_of_pair);
  float* sorted_w = reinterpret_cast<float*>(ws + pl.sorted_w);
  uint16_t* x_sorted = reinterpret_cast<uint16_t*>(ws + pl.x_sorted);
  uint16_t* dy = reinterpret_cast<uint16_t*>(ws + pl.dy);
  uint16_t* dh = reinterpret_cast<uint16_t*>(ws + pl.dh);
  uint16_t* dgu = reinterpret_cast<uint16_t*>(ws + pl.dgu);
  uint16_t* dxs = reinterpret_cast<uint16_t*>(ws + pl.dxs);
  const uint16_t* xb = static_cast<const uint16_t*>(x);
  const uint16_t* doutb = static_cast<const uint16_t*>(dout);

  mark(ctx, L.stream, -1);
  if ((e = launch_permute(L, ids, M, k, E, pb)) != cudaSuccess) return cuda_fail(ctx, e, "permute");
  mark(ctx, L.stream, QARL_STAGE_PERMUTE);
  if ((e = launch_scatter_rows(L, xb, M, H, x_sorted, pb.pos_of_pair, static_cast<int>(k), wts, sorted_w)) != cudaSuccess)
    return cuda_fail(ctx, e, "scatter_rows");
  if ((e = launch_scatter_scale_rows(L, doutb, M, H, dy, pb.pos_of_pair, static_cast<int>(k), wts)) != cudaSuccess)
    return cuda_fail(ctx, e, "scatter_scale_rows");
  if (down_f32 && dwts && (e = launch_pair_dot(L, doutb, down_f32, pb.sorted_pair, P, H, k, dwts)) != cudaSuccess)
    return cuda_fail(ctx, e, "pair_dot");
  mark(ctx, L.stream, QARL_STAGE_BWD_ELEMENTWISE);

  CUresult cu = CUDA_SUCCESS;
  auto gemm = [&](const GemmBf16Args& a, const char* what, int stage) {
    cudaError_t ge = launch_gemm_bf16(L, ctx->encode, a, &cu);
    if (cu != CUDA_SUCCESS) {
      snprintf(ctx->err, sizeof(ctx->err), "cuTensorMapEncodeTiled failed with CUresult %d", static_cast<int>(cu));
      return static_cast<int>(QARL_ERR_CUDA);
    }
    if (ge != cudaSuccess) return cuda_fail(ctx, ge, what);
    mark(ctx, L.stream, stage);
    return static_cast<int>(QARL_OK);
  };
  int rc;
  {  // dH = dy . W2_e
    GemmBf16Args a{};
    a.group = 1;
    a.a = dy;
    a.b = static_cast<const uint16_t*>(w2);  // [E][c = h][j = i]
    a.b_mn_major = true;
    a.Mo = P;
    a.No = I;
    a.Kc = H;
    a.E = E;
    a.offsets = pb.offsets;
    a.c_bf16 = dh;
    if ((rc = gemm(a, "moe_bwd dH", QARL_STAGE_BWD_DX)) != QARL_OK) return rc;
  }
  {  // dW2_e = dy^T h
    GemmBf16Args a{};
    a.group = 2;
    a.a = dy;
    a.a_mn_major = true;
    a.b = static_cast<const uint16_t*>(h);
    a.b_mn_major = true;
    a.Mo = H;
    a.No = I;
    a.E = E;
    a.offsets = pb.offsets;
    a.rows_total = P;
    a.c_f32 = dw2;
    if ((rc = gemm(a, "moe_bwd dW2", QARL_STAGE_BWD_DW)) != QARL_OK) return rc;
  }
  if ((e = launch_swiglu_bwd(L, static_cast<const uint16_t*>(gate_up), dh, P, I, dgu)) != cudaSuccess)
    return cuda_fail(ctx, e, "swiglu_bwd");
  mark(ctx, L.stream, QARL_STAGE_BWD_ELEMENTWISE);
  {  // dXs = dGU . W13_e, stored by flat pair id for the combine
    GemmBf16Args a{};
    a.group = 1;
    a.a = dgu;
    a.b = static_cast<const uint16_t*>(w13);  // [E][c = n][j = h]
    a.b_mn_major = true;
    a.Mo = P;
    a.No = H;
    a.Kc = 2 * I;
    a.E = E;
    a.offsets = pb.offsets;
    a.out_rows = pb.sorted_pair;
    a.c_bf16 = dxs;
    if ((rc = gemm(a, "moe_bwd dXs", QARL_STAGE_BWD_DX)) != QARL_OK) return rc;
  }
  {  // dW13_e = dGU^T x
    GemmBf16Args a{};
    a.group = 2;
    a.a = dgu;
    a.a_mn_major = true;
    a.b = x_sorted;
    a.b_mn_major = true;
    a.Mo = 2 * I;
    a.No = H;
    a.E = E;
    a.offsets = pb.offsets;
    a.rows_total = P;
    a.c_f32 = dw13;
    if ((rc = gemm(a, "moe_bwd dW13", QARL_STAGE_BWD_DW)) != QARL_OK) return rc;
  }
  if ((e = launch_combine(L, dxs, ids, M, k, H, E, static_cast<uint16_t*>(dx))) != cudaSuccess)
    return cuda_fail(ctx, e, "combine");
  mark(ctx, L.stream, QARL_STAGE_COMBINE);
  return QARL_OK;
}

size_t qarl_tbpo_workspace_bytes(int64_t B, int64_t T) {
  if (B < 0 || T < 0) return 0;
  return tbpo_workspace_bytes(B, T);
}

int qarl_tbpo_loss(qarl_ctx* ctx, const float* lp_cur, const float* lp_old_learner, const float* lp_old_sampler,
                   const int64_t* offsets, const float* adv, int64_t B, int64_t T, const qarl_tbpo_params* prm,
                   double* r_seq, double* w_seq, double* j_seq, int32_t* flags, float* grad, double* loss,
                   void* workspace, size_t workspace_bytes, void* stream) {
  NvtxRange nvtx_range("qarl_tbpo_loss");
  if (!ctx || B < 0 || T < 0 || !prm || !loss) return QARL_ERR_INVALID_ARG;
  if (!(prm->cap > 1.0) || prm->eps_h < 0.0 || prm->delta_l < 0.0 || prm->delta_h < 0.0) return QARL_ERR_INVALID_ARG;
  if (B > 0x7FFFFF00ll || T / 2048 > 0x7FFFFF00ll) return QARL_ERR_UNSUPPORTED_SHAPE;
  if (B > 0 && (!offsets || !adv || !r_seq || !w_seq || !j_seq || !flags || !workspace)) return QARL_ERR_INVALID_ARG;
  if (T > 0 && (!lp_cur || !lp_old_learner || !lp_old_sampler)) return QARL_ERR_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(workspace) & 255u) return QARL_ERR_MISALIGNED;
  if (workspace_bytes < tbpo_workspace_bytes(B, T)) return QARL_ERR_WORKSPACE_TOO_SMALL;
  TbpoArgs a{};
  a.lp_cur = lp_cur;
  a.lp_old_learner = lp_old_learner;
  a.lp_old_sampler = lp_old_sampler;
  a.offsets = offsets;
  a.adv = adv;
  a.B = B;
  a.T = T;
  a.eps_h = prm->eps_h;
  a.delta_l = prm->delta_l;
  a.delta_h = prm->delta_h;
  a.cap = prm->cap;
  a.r_seq = r_seq;
  a.w_seq = w_seq;
  a.j_seq = j_seq;
  a.flags = flags;
  a.grad = grad;
  a.loss = loss;
  a.workspace = workspace;
  mark(ctx, static_cast<cudaStream_t>(stream), -1);
  cudaError_t e = launch_tbpo(make_launch(ctx, stream), a);
  mark(ctx, static_cast<cudaStream_t>(stream), QARL_STAGE_TBPO);
  return e == cudaSuccess ? QARL_OK : cuda_fail(ctx, e, "tbpo_loss");
}

int qarl_router_fwd(qarl_ctx* ctx, const void* x, int64_t M, int64_t H, const void* wr, int64_t E, int64_t k,
                    float* logits, int32_t* ids, float* wts, void* stream) {
  NvtxRange nvtx_range("qarl_router_fwd");
  if (!ctx || M < 0 || H <= 0 || E <= 0 || k < 1 || k > 32 || k > E) return QARL_ERR_INVALID_ARG;
  if (H % 8 || E % 8 || E > 1024 || M > 0x7FFFFF00ll) return QARL_ERR_UNSUPPORTED_SHAPE;
  if (M == 0) return QARL_OK;
  if (!x || !wr || !logits || !ids || !wts) return QARL_ERR_INVALID_ARG;
  if (!aligned16(x) || !aligned16(wr) || !aligned16(logits)) return QARL_ERR_MISALIGNED;
  Launch L = make_launch(ctx, stream);
  if (L.gemm_path == 0 && router_fused_applies(E, k)) {  // one launch: selection in the GEMM's epilogue
    CUresult cu = CUDA_SUCCESS;
    mark(ctx, L.stream, -1);
    cudaError_t e = launch_router_fused(L, ctx->encode, static_cast<const uint16_t*>(x), M, H,
                                        static_cast<const uint16_t*>(wr), E, k, logits, ids, wts, &cu);
    if (cu != CUDA_SUCCESS) {
      snprintf(ctx->err, sizeof(ctx->err), "cuTensorMapEncodeTiled failed with CUresult %d", static_cast<int>(cu));
      return QARL_ERR_CUDA;
    }
    if (e != cudaSuccess) return cuda_fail(ctx, e, "router");
    mark(ctx, L.stream, QARL_STAGE_ROUTER);
    return QARL_OK;
  }
  GemmBf16Args a{};
  a.a = static_cast<const uint16_t*>(x);   // A(m, h) = x[m, h]
  a.b = static_cast<const uint16_t*>(wr);  // B(e, h) = W_r[e, h]
  a.Mo = M;
  a.No = E;
  a.Kc = H;
  a.c_f32 = logits;
  CUresult cu = CUDA_SUCCESS;
  mark(ctx, L.stream, -1);
  cudaError_t e = launch_gemm_bf16(L, ctx->encode, a, &cu);
  if (cu != CUDA_SUCCESS) {
    snprintf(ctx->err, sizeof(ctx->err), "cuTensorMapEncodeTiled failed with CUresult %d", static_cast<int>(cu));
    return QARL_ERR_CUDA;
  }
  if (e != cudaSuccess) return cuda_fail(ctx, e, "router logits");
  if ((e = launch_router_topk(L, logits, M, E, k, ids, wts)) != cudaSuccess) return cuda_fail(ctx, e, "router top-k");
  mark(ctx, L.stream, QARL_STAGE_ROUTER);
  return QARL_OK;
}

}  // extern "C"
