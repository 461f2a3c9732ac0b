// Internal declarations shared by the library's translation units (not part of the C ABI).
#pragma once
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_fp8.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <vector>

#include "../../include/qarl.h"

namespace qarl {

constexpr int kBlock = 128;               // 128x128 weight blocks, 1x128 activation groups
constexpr float kAlpha = 448.0f;          // max finite e4m3 (Sec. 2.2)
constexpr float kAmaxFloor = 0x1p-40f;    // all-zero block: amax_c = max(amax, 2^-40)

// Scale of one block and the multiplier used to form the codes (Sec. 2.2, Quant):
// s = fl(amax_c / 448), code = e4m3(fl(x * fl(448 / amax_c))).  IEEE division, no fast math.
__device__ __forceinline__ float block_scale(float amax, float* inv) {
  const float amax_c = fmaxf(amax, kAmaxFloor);
  *inv = __fdiv_rn(kAlpha, amax_c);
  return __fdiv_rn(amax_c, kAlpha);
}

// Two fp32 -> two e4m3 codes (round to nearest even, saturate to +-448); lo in bits [0,8).
__device__ __forceinline__ uint32_t cvt_e4m3x2(float lo, float hi) {
  uint16_t r;
  asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(r) : "f"(hi), "f"(lo));
  return r;
}
__device__ __forceinline__ uint32_t cvt_e4m3x4(float a, float b, float c, float d) {
  return cvt_e4m3x2(a, b) | (cvt_e4m3x2(c, d) << 16);
}

__device__ __forceinline__ float bf16_bits_to_f32(uint32_t bits16) { return __uint_as_float(bits16 << 16); }
// fp32 -> bf16 bits, round to nearest even.
__device__ __forceinline__ uint32_t f32_to_bf16_bits(float f) {
  return static_cast<uint32_t>(__bfloat16_as_ushort(__float2bfloat16_rn(f)));
}
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
  return f32_to_bf16_bits(lo) | (f32_to_bf16_bits(hi) << 16);
}

// Programmatic dependent launch: every kernel of the library is launched so that it may begin
// while its predecessor in the stream is still draining.  A kernel calls pdl_trigger() at once
// (its successor may start launching) and pdl_wait() before its first access to global memory
// (the predecessor, and transitively everything before it, has completed and is visible).
// Only barrier set-up, TMEM allocation and other memory-free preamble runs ahead of the wait.
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// Device status word protocol: first error wins.
__device__ __forceinline__ void set_status(int* status, int code) { atomicCAS(status, 0, code); }

// ---- launchers (host), one per kernel family; every launcher returns a cudaError_t -------
struct Launch {
  cudaStream_t stream;
  int device;
  int sm_count;
  int* d_status;
  int64_t* launches;  // host counter
  unsigned long long wait_limit_ns = 0;  // bound of every device-side barrier wait (0: the default, 2 s)
  int stop_after_stages = -1;            // test harness only: FP8 GEMM producers stop after this many stages
  int gemm_path = 0;                     // test harness only: 0 = automatic, 1 = wide-tile kernel, 2 = decode kernel (one launch per projection)
};

// Launch with the programmatic-stream-serialization attribute (see pdl_wait above).
template <typename... KArgs, typename... Args>
cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, unsigned block, size_t smem, cudaStream_t stream,
                       Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = dim3(block);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

// pub_codes / pub_scales: optional second destination (the copy published to the rollout engine)
cudaError_t launch_quantize_weight(const Launch& L, const uint16_t* w, int64_t E, int64_t N, int64_t K,
                                   uint8_t* codes, float* scales, uint8_t* pub_codes = nullptr,
                                   float* pub_scales = nullptr);
// dst_rows == nullptr: row m of the output is m.  Otherwise each input row t is written to
// the `fanout` output rows dst_rows[t*fanout + j] (quantize once, scatter k times).
// With dst_rows, pair_w [M*fanout] (the top-k weights by flat pair id) is scattered alongside
// into sorted_w[dst] so that later kernels read a pair's weight by its sorted position.
cudaError_t launch_quantize_act(const Launch& L, const uint16_t* x, int64_t M, int64_t K, int64_t ldx,
                                uint8_t* codes, float* scales, const int32_t* dst_rows, int fanout,
                                const float* pair_w = nullptr, float* sorted_w = nullptr);

struct PermuteBuffers {
  int32_t* chunk_hist;   // [nchunks, E]
  int32_t* offsets;      // [E+1]
  int32_t* sorted_pair;  // [P]
  int32_t* pos_of_pair;  // [P]
};
int64_t permute_num_chunks(int64_t P);
cudaError_t launch_permute(const Launch& L, const int32_t* ids, int64_t M, int64_t k, int64_t E,
                           const PermuteBuffers& b);

// Decode-sized layers (M * k <= 2048): the grouping and the scattering activation quantization in one launch.
bool moe_prep_small_applies(int64_t M, int64_t k, int64_t E);
// `zero` / `zero_count`: int32 words the kernel clears (the counters of the one-launch layer that follows).
cudaError_t launch_moe_prep_small(const Launch& L, const int32_t* ids, int64_t M, int64_t k, int64_t E,
                                  const PermuteBuffers& b, const uint16_t* x, int64_t K, const float* pair_w,
                                  uint8_t* codes, float* scales, float* sorted_w, int32_t* zero = nullptr,
                                  int zero_count = 0);

// pos_of_pair == nullptr: contrib is indexed by flat pair id; else by pos_of_pair[pair] (sorted order)
cudaError_t launch_combine(const Launch& L, const uint16_t* contrib, const int32_t* ids, int64_t M, int64_t k,
                           int64_t H, int64_t E, uint16_t* out, const int32_t* pos_of_pair = nullptr);

cudaError_t launch_wait_selftest(const Launch& L, unsigned long long limit_ns);
cudaError_t launch_fp8_mma_peak(const Launch& L, int kblocks);
cudaError_t launch_read_stream(const Launch& L, const void* buf, size_t bytes, uint32_t* sink);
cudaError_t launch_rmsnorm(const Launch& L, const uint16_t* x, int64_t M, int64_t H, float eps, uint16_t* out);

enum GemmMode { kModeLinear = 0, kModeGateUp = 1, kModeDown = 2 };

struct GemmArgs {
  GemmMode mode;
  // A: codes [rows_total, K] (rows = tokens for linear, sorted pairs for MoE) and scales [rows_total, K/128]
  const uint8_t* a_codes;
  const float* a_scales;
  int64_t rows_total;
  int64_t K;
  // B: codes [E, N, K] and scales [E, N/128, K/128]
  const uint8_t* b_codes;
  const float* b_scales;
  int64_t N;
  int64_t E;
  // row groups: expert e owns rows offsets[e] .. offsets[e+1]-1 (device array).  nullptr:
  // one group of rows_total rows (dense).
  const int32_t* offsets;
  // outputs
  uint16_t* out_bf16;        // linear: y [M, N]; gate_up (debug): gate_up [P, 2I]; down: contrib [P, H] by pair id
  float* out_f32;            // optional fp32 accumulator dump (linear: [M,N]; down: [P,H] sorted order)
  uint8_t* h_codes;          // gate_up: [P, I]
  float* h_scales;           // gate_up: [P, I/128]
  uint16_t* h_bf16;          // gate_up (debug): [P, I]
  const int32_t* sorted_pair;   // down: [P]
  const float* pair_weights;    // down: [M*k] by sorted position
};
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
// Returns cudaSuccess, or an error; *cu_err receives a driver error from tensor-map encoding.
cudaError_t launch_gemm(const Launch& L, EncodeTiledFn encode, const GemmArgs& a, CUresult* cu_err);
// The swapped-operand kernel for decode-sized row groups (same bytes out; see gemm_decode_sm100.cu);
// launch_gemm picks it when gemm_decode_applies (L.gemm_path forces one or the other in tests).
bool gemm_decode_applies(const GemmArgs& a);
cudaError_t launch_gemm_decode(const Launch& L, EncodeTiledFn encode, const GemmArgs& a, CUresult* cu_err);
// The decode-sized MoE layer after its grouping / quantization as ONE launch of that kernel: gate_up tiles,
// down tiles (each waiting on a per-expert counter for the h rows it reads) and the k-sum of the
// contributions.  `g` and `d` are the two projections as launch_gemm takes them (same groups);
// `sync` is [2 + 2 E] int32 that must be zero when the kernel starts.  Same bytes as the separate launches.
bool moe_decode_layer_applies(const GemmArgs& g, const GemmArgs& d);
cudaError_t launch_moe_decode_layer(const Launch& L, EncodeTiledFn encode, const GemmArgs& g, const GemmArgs& d,
                                    const int32_t* ids, const int32_t* pos_of_pair, int64_t M, int64_t k, uint16_t* y,
                                    int* sync, CUresult* cu_err);

// ---- W4A16 (4-bit group-quantized weights, bf16 activations) --------------------------------
// 4-bit weight formats (Sec. 2.2): unsigned integer codes with a zero point, or e2m1 floating point
enum W4Format { kFmtInt4 = 0, kFmtE2m1 = 1 };
cudaError_t launch_quantize_weight_w4(const Launch& L, int fmt, const uint16_t* w, int64_t E, int64_t N, int64_t K,
                                      uint8_t* packed, uint16_t* scales, uint8_t* zeros,
                                      uint8_t* pub_packed = nullptr, uint16_t* pub_scales = nullptr,
                                      uint8_t* pub_zeros = nullptr);
// bf16 row t of x [M, H] -> rows dst_rows[t*fanout + j] of out; pair weights scattered alongside.
cudaError_t launch_scatter_rows(const Launch& L, const uint16_t* x, int64_t M, int64_t H, uint16_t* out,
                                const int32_t* dst_rows, int fanout, const float* pair_w, float* sorted_w);

struct GemmW4Args {
  GemmMode mode;
  int fmt;                  // W4Format
  const uint16_t* a_bf16;   // [rows_total, K]
  int64_t rows_total;
  int64_t K;
  const uint8_t* b_packed;  // [E, N, K/2]
  const uint16_t* b_scales; // bf16 bits [E, K/128, N]
  const uint8_t* b_zeros;   // [E, K/128, N] (integer format only)
  int64_t N;
  int64_t E;
  const int32_t* offsets;   // row groups per expert, or nullptr (dense)
  uint16_t* out_bf16;       // linear: y [M, N]; gate_up (debug): gate_up [P, 2I]; down: contrib [P, H] by pair id
  float* out_f32;           // optional fp32 accumulator dump (linear: [M, N]; down: [P, H] sorted order)
  uint16_t* h_bf16;         // gate_up: h [P, I]
  const int32_t* sorted_pair;
  const float* pair_weights;
};
cudaError_t launch_gemm_w4a16(const Launch& L, EncodeTiledFn encode, const GemmW4Args& a, CUresult* cu_err);
// The swapped-operand kernel for decode-sized row groups (same bytes out; see gemm_w4a16_decode_sm100.cu);
// launch_gemm_w4a16 picks it when gemm_w4a16_decode_applies (L.gemm_path forces one or the other in tests).
bool gemm_w4a16_decode_applies(const GemmW4Args& a);
cudaError_t launch_gemm_w4a16_decode(const Launch& L, EncodeTiledFn encode, const GemmW4Args& a, CUresult* cu_err);

// ---- dense bf16 GEMM (full-precision backward): C[i,j] = sum_c A(i,c) B(j,c) ---------------------
struct GemmBf16Args {
  const uint16_t* a;   // K-major: [Mo, Kc] row-major;  MN-major: [Kc, Mo] row-major
  const uint16_t* b;   // K-major: [No, Kc] row-major;  MN-major: [Kc, No] row-major
  bool a_mn_major, b_mn_major;
  int64_t Mo, No, Kc;
  uint16_t* c_bf16;    // [Mo, No] or nullptr
  float* c_f32;        // [Mo, No] or nullptr
  // group = 0: dense.
  // group = 1 (grouped rows): A [Mo = P rows, Kc] K-major in expert-sorted order, B [E, Kc, No] (MN-major) or
  //   [E, No, Kc] (K-major); row p uses the B of the expert that owns it; C [P, No]; Kc % 64 == 0.
  // group = 2 (grouped contraction): A [rows_total, Mo] and B [rows_total, No], both MN-major, expert-sorted
  //   rows; C [E, Mo, No], C_e = sum over the expert's rows of A[p, :]^T B[p, :] (zeros for an empty expert).
  int group = 0;
  const int32_t* offsets = nullptr;  // [E + 1], device
  int64_t E = 1;
  int64_t rows_total = 0;
  const int32_t* out_rows = nullptr;  // group = 1: C row of sorted row p is out_rows[p] (e.g. the flat pair id)
};
cudaError_t launch_gemm_bf16(const Launch& L, EncodeTiledFn encode, const GemmBf16Args& a, CUresult* cu_err);

// element-wise kernels of the MoE layer's backward
cudaError_t launch_scatter_scale_rows(const Launch& L, const uint16_t* dout, int64_t M, int64_t H, uint16_t* dy,
                                      const int32_t* dst_rows, int fanout, const float* pair_w);
cudaError_t launch_swiglu_bwd(const Launch& L, const uint16_t* gate_up, const uint16_t* dh, int64_t P, int64_t I,
                              uint16_t* dgu);
cudaError_t launch_pair_dot(const Launch& L, const uint16_t* dout, const float* y, const int32_t* sorted_pair,
                            int64_t P, int64_t H, int64_t k, float* dwts);

// fp32 logits [M, E] -> top-k ids (descending, ties to the lower id) and softmax weights over the selection
cudaError_t launch_router_topk(const Launch& L, const float* logits, int64_t M, int64_t E, int64_t k, int32_t* ids,
                               float* wts);
// One-launch router (logits tile on the tensor cores, selection and softmax in its epilogue) for E <= 128.
bool router_fused_applies(int64_t E, int64_t k);
cudaError_t launch_router_fused(const Launch& L, EncodeTiledFn encode, const uint16_t* x, int64_t M, int64_t H,
                                const uint16_t* wr, int64_t E, int64_t k, float* logits, int32_t* ids, float* wts,
                                CUresult* cu_err);

// ---- TBPO sequence-level loss ------------------------------------------------------------------
struct TbpoArgs {
  const float* lp_cur;
  const float* lp_old_learner;
  const float* lp_old_sampler;
  const int64_t* offsets;  // [B + 1]
  const float* adv;        // [B]
  int64_t B, T;
  double eps_h, delta_l, delta_h, cap;
  double* r_seq;
  double* w_seq;
  double* j_seq;
  int32_t* flags;
  float* grad;             // [T] or nullptr
  double* loss;
  void* workspace;
};
size_t tbpo_workspace_bytes(int64_t B, int64_t T);
cudaError_t launch_tbpo(const Launch& L, const TbpoArgs& a);

}  // namespace qarl

// The opaque context of the C ABI (one per device).
struct qarl_ctx {
  int device;
  int sm_count;
  int* d_status;
  int64_t launches;
  unsigned long long wait_limit_ns = 0;  // 0: default; set only by the test harness
  int stop_after_stages = -1;            // -1: off; set only by the test harness
  int gemm_path = 0;                     // 0: automatic; set only by the test harness
  qarl::EncodeTiledFn encode;
  char err[256];
  // stage timing: marks[i] closes stage mark_stage[i] (-1: an opening mark)
  std::vector<cudaEvent_t> marks;
  std::vector<int> mark_stage;
  size_t marks_used = 0;
};
