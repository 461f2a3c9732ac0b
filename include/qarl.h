/*
 * qarl.h -- C ABI of the B200-native block-scaled FP8 quantized forward.
 *
 * The library implements the quantized forward that a low-bit rollout decoder and the
 * rollout-aligned training-side forward share (QaRL, Sec. 3.1, components 1 and 2):
 *   Quant (Sec. 2.2, floating-point quantization):  s = max|W| / alpha,  W_q = [W / s]_FP8,
 *                                                    alpha = 448 (e4m3);
 *   low-bit GEMM with rescale (Sec. 2.2):            Y ~= (s_x s_w) (X_q W_q),
 * applied with one fp32 scale per 128x128 weight block and per 1x128 activation group, on
 * dense projections and on the routed-expert FFN (gate_up -> SwiGLU -> re-quantize -> down ->
 * top-k weighted combine).  The K reduction order is fixed (App. C, batch-invariant kernel):
 * every output row is bitwise identical whatever M, batch composition or tile schedule.
 *
 * Conventions for every call
 *   - Every data pointer is a DEVICE pointer owned by the caller; the library never
 *     allocates, frees or keeps caller memory in these calls.  `stream` is a cudaStream_t
 *     passed as void*; all work is enqueued on it and the call returns without synchronizing.
 *   - bf16 tensors are row-major arrays of 16-bit patterns; codes are e4m3 ("fn": no
 *     infinities, max 448) bytes; scales are fp32.
 *   - Pointers to bf16, code and fp32-output tensors must be 16-byte aligned (scale and id
 *     arrays: 4-byte); N, K, H, I must be multiples of 128.  M >= 0 is
 *     arbitrary; M = 0 enqueues nothing and returns QARL_OK.
 *   - Errors the host can see (null pointer, bad shape, misalignment, small workspace) are
 *     returned before anything is launched.  Errors only the device can see (an expert id
 *     outside [0, E), an expert repeated within one token, a bounded wait that expired) set
 *     the context's device status word; the outputs of that call are unspecified and the
 *     error is reported by qarl_poll_device_status.
 *   - A context belongs to one device and may be used from one host thread at a time.  Several
 *     contexts (on the same or on different devices) may be used from several host threads at
 *     once: the little process-wide state the library keeps (per-device launch attributes, the
 *     address of the static scratch array) is written atomically and idempotently.
 *   - There is no CPU fallback: without an sm_100 device qarl_create fails.
 */
#ifndef QARL_H_
#define QARL_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct qarl_ctx qarl_ctx; /* opaque */

typedef enum {
  QARL_OK = 0,
  QARL_ERR_INVALID_ARG = -1,         /* null pointer, negative size, k out of range        */
  QARL_ERR_UNSUPPORTED_SHAPE = -2,   /* N, K, H or I not a multiple of 128, sizes too big  */
  QARL_ERR_MISALIGNED = -3,          /* a pointer or row stride is not 16-byte aligned     */
  QARL_ERR_WORKSPACE_TOO_SMALL = -4,
  QARL_ERR_UNSUPPORTED_DEVICE = -5,  /* not compute capability 10.x                        */
  QARL_ERR_CUDA = -6,                /* a CUDA runtime / driver call failed                */
  QARL_ERR_DEVICE_TIMEOUT = -7,      /* a bounded device-side wait expired                 */
  QARL_ERR_BAD_EXPERT_ID = -8        /* id outside [0,E) or repeated within a token        */
} qarl_status;

/* Create a context on CUDA device `device` (host call; allocates a few bytes of device
 * memory for the status word).  Fails with QARL_ERR_UNSUPPORTED_DEVICE unless the device
 * has compute capability 10.x.  *out is set to NULL on failure. */
int qarl_create(qarl_ctx** out, int device);
void qarl_destroy(qarl_ctx* ctx);
/* Static string for a status code (never NULL). */
const char* qarl_status_string(int status);
/* Synchronizes `stream`, then returns and clears the device status word (QARL_OK if no
 * device-side error was recorded since the last poll). */
int qarl_poll_device_status(qarl_ctx* ctx, void* stream);
/* Text of the last CUDA error the context saw (host memory owned by the context). */
const char* qarl_last_cuda_error(qarl_ctx* ctx);

/* Sec. 2.2 Quant, 128x128 blocks (Sec. 3.1 item 2: done on the fly from the bf16 masters).
 * in : w_bf16  device bf16 [E, N, K] row-major (E = 1 for a dense weight).
 * out: codes   device u8   [E, N, K];  scales device f32 [E, N/128, K/128].
 * Per block: amax = max|w|, s = max(amax, 2^-40) / 448, code = e4m3_rne_sat(w * (448 / max(amax, 2^-40))). */
int qarl_quantize_weight(qarl_ctx* ctx, const void* w_bf16, int64_t E, int64_t N, int64_t K,
                         uint8_t* codes, float* scales, void* stream);

/* The same quantization, fused with publishing (Sec. 3.1 item 3: the low-bit tensors the
 * training forward has just materialised are handed to the rollout engine as they are, with no
 * second quantization pass).  pub_codes / pub_scales: a second destination of the same shapes,
 * written from the same registers in the same launch -- the rollout engine's weight buffers:
 * device memory of this GPU or peer-mapped memory of another one (plain stores).  Both NULL:
 * identical to qarl_quantize_weight.  The two copies are bitwise equal by construction. */
int qarl_quantize_weight_publish(qarl_ctx* ctx, const void* w_bf16, int64_t E, int64_t N, int64_t K,
                                 uint8_t* codes, float* scales, uint8_t* pub_codes,
                                 float* pub_scales, void* stream);

/* Sec. 2.2 Quant, 1x128 groups along K.
 * in : x_bf16 device bf16 [M, K] with row stride ldx elements (ldx >= K, ldx % 8 == 0).
 * out: codes  device u8 [M, K] (dense);  scales device f32 [M, K/128]. */
int qarl_quantize_act(qarl_ctx* ctx, const void* x_bf16, int64_t M, int64_t K, int64_t ldx,
                      uint8_t* codes, float* scales, void* stream);

/* Sec. 2.2 low-bit GEMM with rescale, per 128-wide K-block:
 *   y[m,n] = bf16( sum_kb  fl(s_x[m,kb] * s_w[n/128,kb]) * (x_q[m,kb,:] . w_q[n,kb,:]) ),
 * fp32 accumulation, kb ascending, starting from 0 (fixed order, App. C).
 * qarl_linear_fwd quantizes x first (as qarl_quantize_act) into `workspace`;
 * qarl_linear_fwd_q takes activations that are already quantized.
 * in : x_bf16 [M, K] dense;  w_codes [N, K], w_scales [N/128, K/128] from qarl_quantize_weight.
 * out: y_bf16 [M, N];  y_f32 optional (may be NULL) fp32 copy of the accumulator [M, N].
 * workspace: device scratch of at least qarl_linear_workspace_bytes(M, N, K) bytes, 256-byte
 * aligned; its contents are undefined afterwards.  Calls that share a workspace must not
 * overlap on the device. */
size_t qarl_linear_workspace_bytes(int64_t M, int64_t N, int64_t K);
int qarl_linear_fwd(qarl_ctx* ctx, const void* x_bf16, int64_t M, int64_t K,
                    const uint8_t* w_codes, const float* w_scales, int64_t N,
                    void* y_bf16, float* y_f32, void* workspace, size_t workspace_bytes,
                    void* stream);
int qarl_linear_fwd_q(qarl_ctx* ctx, const uint8_t* x_codes, const float* x_scales,
                      int64_t M, int64_t K, const uint8_t* w_codes, const float* w_scales,
                      int64_t N, void* y_bf16, float* y_f32, void* stream);

/* Allocation-free variant of qarl_linear_fwd (the paper has no counterpart; this is a
 * packaging choice of this library).
 *
 * Who needs it: code that is not allowed to obtain device memory when it makes the call -- a
 * serving process that handed every free byte of the GPU to its KV-cache pool at start-up, a
 * plugin running under a host application that owns the allocator, a latency-critical loop
 * in which cudaMalloc's implicit device synchronization is unacceptable.  Such a caller
 * cannot hand over the workspace qarl_linear_fwd asks for.  Here the scratch (the e4m3 copy of
 * the activations and their scales) is a fixed array inside the library's device image instead:
 * QARL_STATIC_LINEAR_MAX_ELEMS bytes of codes plus 1/32 of that for scales (about 4.1 MiB),
 * resident on every GPU that loads the library, for the life of the process.
 *
 * Same arithmetic and same output bytes as qarl_linear_fwd.  The caller still passes the
 * input and the output: x_bf16 [M, K] dense, w_codes [N, K], w_scales [N/128, K/128], y_bf16
 * [M, N] (device pointers, alignment as for qarl_linear_fwd); there is no fp32 dump.
 *   - M * K must not exceed QARL_STATIC_LINEAR_MAX_ELEMS, otherwise the call returns
 *     QARL_ERR_UNSUPPORTED_SHAPE before launching anything (qarl_last_cuda_error has the text).
 *   - The call performs no cudaMalloc / cudaFree and calls no allocating library routine.
 *   - The first call on a device looks up the array's device address; the context's device
 *     must be the current device for that call, and that first call should be made before
 *     any stream capture begins.
 *   - All calls on a device share the one array, which keeps whatever the last call left in
 *     it.  Every byte a call reads it has first rewritten itself, so nothing needs clearing
 *     between calls; but two calls that overlap on the GPU (different streams, or different
 *     contexts on the same device) race on the array and corrupt each other's results. */
#define QARL_STATIC_LINEAR_MAX_ELEMS (4 * 1024 * 1024)
int qarl_linear_fwd_static(qarl_ctx* ctx, const void* x_bf16, int64_t M, int64_t K,
                           const uint8_t* w_codes, const float* w_scales, int64_t N,
                           void* y_bf16, void* stream);

/* Optional dumps of the MoE layer's intermediates (every field may be NULL).  "Sorted
 * order" is the order of token-expert pairs after grouping by expert: position q holds the
 * flat pair sorted_pair[q] = t*k + j. */
typedef struct {
  int32_t* expert_offsets; /* [E+1]  first sorted position of each expert; [E] = M*k      */
  int32_t* sorted_pair;    /* [M*k]  pairs stably sorted by expert id (ties by pair id)    */
  void* gate_up_bf16;      /* [M*k, 2I] sorted order, bf16 of the gate_up accumulator      */
  void* h_bf16;            /* [M*k, I]  sorted order, bf16( silu(gate) * up )              */
  uint8_t* h_codes;        /* [M*k, I]  sorted order                                       */
  float* h_scales;         /* [M*k, I/128] sorted order                                    */
  float* down_f32;         /* [M*k, H]  sorted order, fp32 accumulator of the down GEMM    */
} qarl_moe_debug;

/* One routed-expert FFN layer on quantized weights (Sec. 3.1 items 1-2 applied to the MoE
 * block; the paper notes MoE decode is memory-bound, App. D.1).  For every token t and slot j
 * with expert e = topk_ids[t,j]:
 *   x_q = quantize_act(x[t]);  gu = bf16(blockscaled(x_q, W13_e));  h = bf16(silu(gu[:I]) * gu[I:]);
 *   h_q = quantize_act(h);     y = blockscaled(h_q, W2_e) (fp32);   c_j = bf16(topk_weights[t,j] * y);
 *   out[t] = bf16( sum of float(c_j) over the token's slots in ASCENDING EXPERT ID, from 0 ).
 * in : x_bf16 [M, H];  topk_ids i32 [M, k];  topk_weights f32 [M, k] (used as given);
 *      w13_codes [E, 2I, H] (rows 0..I-1 gate, I..2I-1 up; scale blocks over the whole
 *      [2I, H] matrix), w13_scales [E, 2I/128, H/128];  w2_codes [E, H, I], w2_scales [E, H/128, I/128].
 * out: out_bf16 [M, H].
 * Limits: 1 <= k <= 32, 1 <= E <= 1024, M*k < 2^31.
 * workspace: at least qarl_moe_workspace_bytes(M, H, I, E, k) bytes, 256-byte aligned; the
 * call clears what must start at zero; calls sharing a workspace must not overlap.
 * Launches: training-sized batches run the steps as separate kernels (grouping, activation
 * quantization, gate_up, down, combine).  Decode-sized batches (M*k <= 2048 and M*k <= 32*E) run
 * two: the grouping with the quantization, then the whole layer as one persistent kernel whose
 * CTAs publish finished tiles to one another through counters in the workspace (every wait on
 * them is bounded like the pipeline waits; expiry gives QARL_ERR_DEVICE_TIMEOUT).  The bytes of
 * out_bf16 and of every dump are the same on both routes. */
size_t qarl_moe_workspace_bytes(int64_t M, int64_t H, int64_t I, int64_t E, int64_t k);
int qarl_moe_fwd(qarl_ctx* ctx, const void* x_bf16, const int32_t* topk_ids,
                 const float* topk_weights, int64_t M, int64_t H, int64_t I, int64_t E,
                 int64_t k, const uint8_t* w13_codes, const float* w13_scales,
                 const uint8_t* w2_codes, const float* w2_scales, void* out_bf16,
                 void* workspace, size_t workspace_bytes, const qarl_moe_debug* dbg,
                 void* stream);

/* ---------------------------------------------------------------------------------------
 * Expert-parallel form of qarl_moe_fwd: the layer cut into the three stages between which rows
 * travel when the experts are split across GPUs (contiguous ranges of expert ids per GPU).
 *   token's GPU : qarl_moe_dispatch      rows quantized once, laid out sorted by expert id
 *   (exchange 1 : each GPU receives the rows of its experts, per source in expert order)
 *   expert's GPU: qarl_moe_experts_fwd   gate_up, SwiGLU, re-quantization, down, * pair weight
 *   (exchange 2 : the bf16 contributions travel back to where their rows came from)
 *   token's GPU : qarl_moe_combine_sorted  the k-sum in ascending expert id
 * The stages run the kernels of qarl_moe_fwd on the same per-row data, so by the row invariance
 * (App. C) the output is bitwise that of qarl_moe_fwd with all experts on one GPU, for any
 * number of GPUs and any split of the tokens.  The exchanges are the caller's (the Python
 * package does them with all-to-all collectives); with one GPU the three calls in a row are the
 * whole layer.  All pointers are device pointers; nothing is allocated.
 * ------------------------------------------------------------------------------------- */

/* in : x_bf16 [M, H], topk_ids [M, k] (global expert ids in [0, E)), topk_weights [M, k] fp32.
 * out: codes_sorted u8 [M*k, H] and scales_sorted fp32 [M*k, H/128]: the quantized row of pair
 *      p's token at position pos_of_pair[p]; weights_sorted fp32 [M*k]: the pair's top-k weight
 *      at the same position; offsets i32 [E+1]: positions [offsets[e], offsets[e+1]) belong to
 *      expert e (stable order of flat pair id inside); pos_of_pair i32 [M*k].
 * workspace: qarl_moe_dispatch_workspace_bytes(M, E, k) bytes, 256-byte aligned.
 * Limits: H % 128 == 0, 1 <= k <= 32, 1 <= E <= 1024, M*k < 2^31.  M == 0: offsets zeroed. */
size_t qarl_moe_dispatch_workspace_bytes(int64_t M, int64_t E, int64_t k);
int qarl_moe_dispatch(qarl_ctx* ctx, const void* x_bf16, const int32_t* topk_ids,
                      const float* topk_weights, int64_t M, int64_t H, int64_t E, int64_t k,
                      uint8_t* codes_sorted, float* scales_sorted, float* weights_sorted,
                      int32_t* offsets, int32_t* pos_of_pair, void* workspace,
                      size_t workspace_bytes, void* stream);

/* in : R rows (codes u8 [R, H], scales fp32 [R, H/128], row_weights fp32 [R]) grouped by local
 *      expert: rows [offsets[j], offsets[j+1]) use expert j of the E_local experts whose weights
 *      are given (w13 [E_local, 2I, H], w2 [E_local, H, I], codes + block scales as
 *      qarl_quantize_weight writes them); offsets i32 [E_local+1] on the device, offsets[E_local] == R.
 * out: contrib bf16 [R, H]: row r = bf16(row_weights[r] * (h_r . W2_e)), in the order of the input.
 * workspace: qarl_moe_experts_workspace_bytes(R, I) bytes, 256-byte aligned.
 * Limits: H % 128 == 0, I % 128 == 0, 1 <= E_local <= 1024, R < 2^31. */
size_t qarl_moe_experts_workspace_bytes(int64_t R, int64_t I);
int qarl_moe_experts_fwd(qarl_ctx* ctx, const uint8_t* codes, const float* scales,
                         const float* row_weights, const int32_t* offsets, int64_t R, int64_t H,
                         int64_t I, int64_t E_local, const uint8_t* w13_codes,
                         const float* w13_scales, const uint8_t* w2_codes, const float* w2_scales,
                         void* contrib_bf16, void* workspace, size_t workspace_bytes, void* stream);

/* out[t] = bf16(sum over the token's k pairs, in ascending expert id, of
 * float(contrib_sorted[pos_of_pair[t*k + j]])), starting from 0.0f: the last step of
 * qarl_moe_fwd on contributions held in dispatch order.  contrib_sorted bf16 [M*k, H];
 * topk_ids and pos_of_pair as given to / written by qarl_moe_dispatch.  H % 8 == 0. */
int qarl_moe_combine_sorted(qarl_ctx* ctx, const void* contrib_sorted_bf16, const int32_t* topk_ids,
                            const int32_t* pos_of_pair, int64_t M, int64_t H, int64_t E, int64_t k,
                            void* out_bf16, void* stream);

/* ---------------------------------------------------------------------------------------
 * W4A16: 4-bit integer weight-only quantization with bf16 activations (Sec. 2.2, integer
 * quantization: W_q = clamp(round(W/s) + z, q_min, q_max), W^ = s (W_q - z); Sec. 3.1 item 1
 * names W4A16 as the format of the larger MoE models).  Choices the paper leaves open, fixed
 * here: unsigned codes 0..15; one (s, z) per 128 consecutive K elements of one weight row;
 * lo = min(0, min W), hi = max(0, max W); s = bf16(max(hi - lo, 2^-40) / 15);
 * z = clamp(rint(-lo / s), 0, 15); round = nearest, ties to even; the GEMM multiplies bf16
 * activations by w^ = bf16(s * (W_q - z)) and accumulates in fp32 in ascending k.
 *
 * Storage (all device pointers):
 *   packed  u8, E*N*K/2 bytes, tile-major: the codes of weight rows [128b, 128b+128) x K
 *                             elements [64c, 64c+64) of expert e form the contiguous 4096-byte
 *                             chunk number (e*(N/128) + b)*(K/64) + c.  Inside a chunk the
 *                             32-bit word w (0..7, eight consecutive codes e0..e7 each) of row
 *                             r sits at byte (w/4)*2048 + r*16 + (w%4)*4; inside a word the
 *                             codes lie nibble by nibble from the low end in the order
 *                             e0 e2 e4 e6 e1 e3 e5 e7 (so bits [4j, 4j+4) and [16+4j, 20+4j)
 *                             hold the adjacent pair e_2j, e_2j+1);
 *   scales  bf16 [E, K/128, N]  group-major: the scales of one K-group for all rows of an
 *                             expert are contiguous;
 *   zeros   u8  [E, K/128, N]  same layout.
 * ------------------------------------------------------------------------------------- */

/* in : w_bf16 [E, N, K], 16-byte aligned, N % 128 == 0, K % 128 == 0.  out: packed (16-byte aligned),
 * scales (2-byte aligned), zeros, as above; caller-owned.  One kernel, every input byte read once. */
int qarl_quantize_weight_w4(qarl_ctx* ctx, const void* w_bf16, int64_t E, int64_t N, int64_t K,
                            uint8_t* packed, void* scales_bf16, uint8_t* zeros, void* stream);
/* The same, fused with publishing (Sec. 3.1 item 3): pub_* is a second destination of the same
 * shapes (the rollout engine's buffers), written from the same registers in the same launch;
 * all three NULL: identical to qarl_quantize_weight_w4.  The copies are bitwise equal. */
int qarl_quantize_weight_w4_publish(qarl_ctx* ctx, const void* w_bf16, int64_t E, int64_t N,
                                    int64_t K, uint8_t* packed, void* scales_bf16, uint8_t* zeros,
                                    uint8_t* pub_packed, void* pub_scales_bf16, uint8_t* pub_zeros,
                                    void* stream);

/* y[m, n] = bf16( sum_k x[m,k] * w^[n,k] ), fp32 accumulation (Sec. 2.2 Dequant applied inside
 * the GEMM).  in: x_bf16 [M, K] 16-byte aligned; weights as produced by qarl_quantize_weight_w4
 * with E = 1;  N % 128 == 0, K % 128 == 0.  out: y_bf16 [M, N]; y_f32 [M, N] optional (NULL:
 * skipped) dump of the fp32 accumulator.  Needs no workspace.  Row m of y depends only on row m
 * of x and on the weights (App. C): bitwise the same for any M. */
int qarl_linear_fwd_w4a16(qarl_ctx* ctx, const void* x_bf16, int64_t M, int64_t K,
                          const uint8_t* w_packed, const void* w_scales_bf16,
                          const uint8_t* w_zeros, int64_t N, void* y_bf16, float* y_f32,
                          void* stream);

/* The routed-expert FFN layer of qarl_moe_fwd on W4A16 weights; activations stay bf16:
 *   gu = bf16(x[t] . W13^_e);  h = bf16(silu(gu[:I]) * gu[I:]);  y = h . W2^_e (fp32);
 *   c_j = bf16(topk_weights[t,j] * y);  out[t] = bf16(sum of float(c_j) in ascending expert id).
 * w13: [E, 2I, H] quantized along H (rows 0..I-1 gate, I..2I-1 up); w2: [E, H, I] quantized
 * along I.  Limits: H % 256 == 0, I % 128 == 0, 1 <= k <= 32, 1 <= E <= 1024, M*k < 2^31.
 * dbg: expert_offsets, sorted_pair, gate_up_bf16, h_bf16 and down_f32 are filled when non-NULL;
 * h_codes and h_scales are not used.  workspace: at least
 * qarl_moe_w4a16_workspace_bytes(M, H, I, E, k) bytes, 256-byte aligned; calls sharing a
 * workspace must not overlap.  Errors as qarl_moe_fwd. */
size_t qarl_moe_w4a16_workspace_bytes(int64_t M, int64_t H, int64_t I, int64_t E, int64_t k);
int qarl_moe_fwd_w4a16(qarl_ctx* ctx, const void* x_bf16, const int32_t* topk_ids,
                       const float* topk_weights, int64_t M, int64_t H, int64_t I, int64_t E,
                       int64_t k, const uint8_t* w13_packed, const void* w13_scales_bf16,
                       const uint8_t* w13_zeros, const uint8_t* w2_packed,
                       const void* w2_scales_bf16, const uint8_t* w2_zeros, void* out_bf16,
                       void* workspace, size_t workspace_bytes, const qarl_moe_debug* dbg,
                       void* stream);

/* ---------------------------------------------------------------------------------------
 * FP4A16: e2m1 floating-point weight-only quantization with bf16 activations (Sec. 2.2,
 * floating-point quantization: s = max|W| / alpha, W_q = [W / s]_FP4, W^ = s W_q, alpha = 6, the
 * largest finite e2m1 value).  A code is sign (bit 3) | two exponent bits (bias 1) | one mantissa
 * bit: magnitudes 0, .5, 1, 1.5, 2, 3, 4, 6; no infinity, no NaN.  Choices the paper leaves
 * open, fixed here as for the integer format: one s per 128 consecutive K elements of one weight
 * row; s = bf16(max(amax, 2^-40) / 6); W / s is the IEEE fp32 quotient; [.]_FP4 rounds to the
 * nearest value, ties to the even code, saturating at +-6; the sign bit is that of W (also on
 * zero); the GEMM multiplies bf16 activations by w^ = bf16(s * value) and accumulates in fp32 in
 * ascending k.  Storage: packed and scales exactly as for W4A16 above (same tile-major chunks,
 * same nibble order, bf16 scales [E, K/128, N]); there are no zero points.
 * ------------------------------------------------------------------------------------- */

/* in : w_bf16 [E, N, K], 16-byte aligned, N % 128 == 0, K % 128 == 0.  out: packed (16-byte
 * aligned), scales (2-byte aligned); caller-owned.  pub_packed / pub_scales_bf16: optional second
 * destination written in the same launch (Sec. 3.1 item 3: the rollout engine's copy), both NULL
 * or both set.  One kernel, every input byte read once.  Errors as qarl_quantize_weight_w4. */
int qarl_quantize_weight_fp4(qarl_ctx* ctx, const void* w_bf16, int64_t E, int64_t N, int64_t K,
                             uint8_t* packed, void* scales_bf16, uint8_t* pub_packed,
                             void* pub_scales_bf16, void* stream);

/* qarl_linear_fwd_w4a16 on e2m1 weights (E = 1): same shapes, limits, outputs, row invariance. */
int qarl_linear_fwd_fp4a16(qarl_ctx* ctx, const void* x_bf16, int64_t M, int64_t K,
                           const uint8_t* w_packed, const void* w_scales_bf16, int64_t N,
                           void* y_bf16, float* y_f32, void* stream);

/* qarl_moe_fwd_w4a16 on e2m1 weights: same computation, limits, debug outputs and workspace
 * (qarl_moe_w4a16_workspace_bytes). */
int qarl_moe_fwd_fp4a16(qarl_ctx* ctx, const void* x_bf16, const int32_t* topk_ids,
                        const float* topk_weights, int64_t M, int64_t H, int64_t I, int64_t E,
                        int64_t k, const uint8_t* w13_packed, const void* w13_scales_bf16,
                        const uint8_t* w2_packed, const void* w2_scales_bf16, void* out_bf16,
                        void* workspace, size_t workspace_bytes, const qarl_moe_debug* dbg,
                        void* stream);

/* ---------------------------------------------------------------------------------------
 * Training-side backward of a quantized linear layer y = x . W^T (Sec. 3.1 item 2: the forward
 * runs on Quant(W), the backward in full precision; the straight-through estimator treats Quant
 * as the identity and the gradients belong to the bf16 master weights):
 *   dX[m,k] = sum_n dY[m,n] W[n,k]  -> dx_bf16 [M, K] (and dx_f32 [M, K] if not NULL)
 *   dW[n,k] = sum_m dY[m,n] X[m,k]  -> dw_f32 [N, K] (fp32, overwritten, not accumulated)
 * in : dy_bf16 [M, N], x_bf16 [M, K], w_bf16 [N, K] (the masters, not the codes); device
 *      pointers, 16-byte aligned; N % 8 == 0, K % 8 == 0, M >= 1.  Either output group may be
 *      skipped: dx_bf16 == NULL && dx_f32 == NULL skips dX, dw_f32 == NULL skips dW.
 * Two launches of one bf16 tensor-core GEMM that reads its operands in either orientation, so
 * no transposed copy is made; fp32 accumulation in one fixed order (ascending n, resp. m): a
 * row of dX depends only on that row of dY.  Needs no workspace. */
int qarl_linear_bwd(qarl_ctx* ctx, const void* dy_bf16, const void* x_bf16, const void* w_bf16,
                    int64_t M, int64_t N, int64_t K, void* dx_bf16, float* dx_f32, float* dw_f32,
                    void* stream);

/* The same backward for an expert projection of the MoE layer, on the forward's expert-sorted row
 * layout (expert e owns rows offsets[e] .. offsets[e+1]-1 of dy and x; offsets i32 [E+1] on the
 * device, as qarl_moe_fwd's debug output expert_offsets gives them):
 *   dX[p, k]   = sum_n dY[p, n] W_e[n, k]   for the expert e that owns row p   -> dx_bf16 / dx_f32 [P, K]
 *   dW_e[n, k] = sum over the expert's rows p of dY[p, n] X[p, k]              -> dw_f32 [E, N, K]
 * in : dy_bf16 [P, N], x_bf16 [P, K], w_bf16 [E, N, K] (masters); N % 64 == 0, K % 8 == 0,
 *      1 <= E <= 1024.  An expert without rows gets dW_e = 0.  Outputs may be skipped as in
 * qarl_linear_bwd.  No padding, no copies, no workspace; fixed accumulation order (a row of dX
 * depends only on that row of dY; dW_e adds its rows in sorted order). */
int qarl_grouped_linear_bwd(qarl_ctx* ctx, const void* dy_bf16, const void* x_bf16,
                            const void* w_bf16, const int32_t* offsets, int64_t P, int64_t N,
                            int64_t K, int64_t E, void* dx_bf16, float* dx_f32, float* dw_f32,
                            void* stream);

/* Full-precision backward of the routed-expert FFN layer of qarl_moe_fwd (Sec. 3.1 item 2): the
 * straight-through estimator passes the gradient through both quantizers, so the backward runs on
 * the bf16 masters and on the bf16 activations the low-bit forward produced:
 *   dy[q]   = bf16(topk_weights[pair] * dout[token])              per expert-sorted pair q
 *   dH      = bf16(dy . W2_e)          dW2_e  = dy^T h            (fp32)
 *   dGU     = SwiGLU backward of dH on the saved gate / up        (bf16)
 *   dXs     = bf16(dGU . W13_e)        dW13_e = dGU^T x           (fp32)
 *   dx[t]   = bf16(sum of the token's k rows of dXs in ascending expert id)
 *   d_topk_weights[t, j] = <dout[t], y[q]>   (only if down_f32 and d_topk_weights are given)
 * in : x_bf16 [M, H], topk_ids [M, k], topk_weights [M, k], w13_bf16 [E, 2I, H], w2_bf16 [E, H, I]
 *      (masters), gate_up_bf16 [M*k, 2I] and h_bf16 [M*k, I] in expert-sorted order (the forward's
 *      debug outputs of those names), dout_bf16 [M, H]; optional down_f32 [M*k, H] sorted.
 * out: dx_bf16 [M, H], dw13_f32 [E, 2I, H], dw2_f32 [E, H, I] (overwritten; zeros for an expert
 *      without tokens), optional d_topk_weights f32 [M, k].
 * Limits as qarl_moe_fwd, and H % 64 == 0, I % 32 == 0.
 * workspace: qarl_moe_bwd_workspace_bytes(M, H, I, E, k) bytes, 256-byte aligned. */
size_t qarl_moe_bwd_workspace_bytes(int64_t M, int64_t H, int64_t I, int64_t E, int64_t k);
int qarl_moe_bwd(qarl_ctx* ctx, const void* x_bf16, const int32_t* topk_ids,
                 const float* topk_weights, int64_t M, int64_t H, int64_t I, int64_t E, int64_t k,
                 const void* w13_bf16, const void* w2_bf16, const void* gate_up_bf16,
                 const void* h_bf16, const void* dout_bf16, const float* down_f32, void* dx_bf16,
                 float* dw13_f32, float* dw2_f32, float* d_topk_weights, void* workspace,
                 size_t workspace_bytes, void* stream);

/* ---------------------------------------------------------------------------------------
 * TBPO: the sequence-level surrogate of Sec. 3.2 over B packed responses (ratio and weight as
 * written out in the appendix "Detail of TBPO").  Response i owns tokens
 * [offsets[i], offsets[i+1]) of the flat arrays (offsets monotone, offsets[0] = 0,
 * offsets[B] = T; prompt and padding tokens are simply not in the arrays).  With L its length:
 *   a = (1/L) sum_t (lp_cur - lp_old_learner)[t]          r = exp(a)    r_seq-prox
 *   b = (1/L) sum_t (lp_old_learner - lp_old_sampler)[t]  w = exp(b)    w_seq-mismatch
 *   w~ = exp(clip(b, -log cap, log cap))                  (two-sided cap, taken in the log domain)
 *   r~ = clip(r, 0, 1 + eps_h)            if adv[i] >= 0
 *        clip(r, 1 - delta_l, 1 + delta_h) if adv[i] <  0
 *   J = w~ r~ adv[i];   loss = -(1/B) sum_i J;
 *   grad[t] = d loss / d lp_cur[t] = -(w~ adv r) / (L B) if r lies inside its band (bounds
 *   inclusive), else 0: a response outside its band is masked from the update.
 * An empty response has r = w = 1, J = 0 and counts in B.  All arithmetic in double on the fp32
 * inputs, every sum in a fixed order (results do not depend on the grid).
 * in : lp_* f32 [T], offsets i64 [B+1], adv f32 [B]: device pointers.  params: host struct
 *      (the paper's table: eps_h 4e-4, delta_l 3e-4, delta_h 7e-4, cap 2).
 * out: r_seq, w_seq, j_seq f64 [B]; flags i32 [B] (bit 0: r outside its band, bit 1: w capped,
 *      bit 2: empty); grad f32 [T] (NULL: skipped); loss f64 [1]: device pointers, caller-owned.
 * workspace: qarl_tbpo_workspace_bytes(B, T) bytes, 256-byte aligned. */
typedef struct {
  double eps_h, delta_l, delta_h, cap;
} qarl_tbpo_params;
size_t qarl_tbpo_workspace_bytes(int64_t B, int64_t T);
int qarl_tbpo_loss(qarl_ctx* ctx, const float* lp_cur, const float* lp_old_learner,
                   const float* lp_old_sampler, const int64_t* offsets, const float* adv, int64_t B,
                   int64_t T, const qarl_tbpo_params* params, double* r_seq, double* w_seq,
                   double* j_seq, int32_t* flags, float* grad, double* loss, void* workspace,
                   size_t workspace_bytes, void* stream);

/* ---------------------------------------------------------------------------------------
 * Router of the MoE block (the paper names the "router shift" between sampler and learner,
 * Sec. 4.2, but gives no formula; this is the top-k softmax router of the model family it
 * trains).  The router is not quantized:
 *   logits[m, e] = sum_h x[m, h] W_r[e, h]   bf16 operands, fp32 accumulation in a fixed order
 *   topk_ids[m, :]     the k largest logits of token m in descending order, ties to the lower id
 *   topk_weights[m, :] softmax over those k logits (fp32)
 * in : x_bf16 [M, H], w_router_bf16 [E, H]: device, 16-byte aligned; H % 8 == 0, E % 8 == 0,
 *      E <= 1024, 1 <= k <= min(E, 32).
 * out: logits_f32 [M, E] (required), topk_ids i32 [M, k], topk_weights f32 [M, k]; caller-owned.
 *      The outputs feed qarl_moe_fwd directly.
 * Up to 128 experts and k <= 16 the call is one launch (the selection runs in the epilogue of the
 * logits GEMM); beyond that two (GEMM, then a selection kernel).  Both give the same bytes.
 * A token's routing depends only on that token's row of x: bitwise the same for any M. */
int qarl_router_fwd(qarl_ctx* ctx, const void* x_bf16, int64_t M, int64_t H,
                    const void* w_router_bf16, int64_t E, int64_t k, float* logits_f32,
                    int32_t* topk_ids, float* topk_weights, void* stream);

/* Tracing: every entry point that launches kernels opens an NVTX range named after itself for the
 * duration of the host call (header-only NVTX 3; a pointer check when no tool is attached), so a
 * timeline profiler shows the library's calls among the caller's own ranges. */

/* Stage timing (measurement aid, no paper counterpart).  Between qarl_profile_begin and
 * qarl_profile_end every call of this context brackets each of its kernels with CUDA events
 * on the caller's stream (events are created in qarl_profile_begin, none in the hot calls;
 * at most max_marks events are used, later kernels go untimed).  qarl_profile_end
 * synchronizes the device, adds the elapsed milliseconds and the number of timed launches of
 * each stage into stage_ms[QARL_NUM_STAGES] / stage_launches[QARL_NUM_STAGES] (host arrays)
 * and destroys the events. */
enum {
  QARL_STAGE_QUANT_WEIGHT = 0,
  QARL_STAGE_QUANT_ACT = 1,   /* W4A16 MoE: the copy of the bf16 rows into expert-sorted order */
  QARL_STAGE_LINEAR_GEMM = 2,
  QARL_STAGE_PERMUTE = 3,
  QARL_STAGE_GATE_UP_GEMM = 4,
  QARL_STAGE_DOWN_GEMM = 5,
  QARL_STAGE_COMBINE = 6,
  QARL_STAGE_BWD_DX = 7,
  QARL_STAGE_BWD_DW = 8,
  QARL_STAGE_TBPO = 9,
  QARL_STAGE_ROUTER = 10,
  QARL_STAGE_BWD_ELEMENTWISE = 11,
  QARL_STAGE_MOE_DECODE_LAYER = 12, /* decode-sized qarl_moe_fwd: gate_up + down + combine in one launch */
  QARL_NUM_STAGES = 13
};
int qarl_profile_begin(qarl_ctx* ctx, int max_marks);
int qarl_profile_end(qarl_ctx* ctx, double* stage_ms, int64_t* stage_launches);

/* Number of this library's kernels the context has launched since it was created. */
int64_t qarl_launch_count(qarl_ctx* ctx);

#ifdef __cplusplus
}
#endif
#endif /* QARL_H_ */
