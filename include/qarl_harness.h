/*
 * qarl_harness.h -- test-harness helpers that ship in the same library but are NOT part of the
 * quantized-forward API.  The paper's pipeline has no counterpart for them: they exist so that
 * the rollout-alignment stack test (consecutive MoE layers with RMSNorm + residual in between)
 * can glue layers together with an operation whose result for a row does not depend on the
 * batch it runs in.
 */
#ifndef QARL_HARNESS_H_
#define QARL_HARNESS_H_

#include "qarl.h"

#ifdef __cplusplus
extern "C" {
#endif

/* out[m,:] = bf16( x[m,:] * rsqrt(mean(x[m,:]^2) + eps) ), weight = 1.  x, out: device bf16
 * [M, H], H a multiple of 8, 16-byte aligned, may alias.  The sum of squares of a row is
 * accumulated in fp32 in a fixed per-row order (lane-strided partial sums, then a butterfly),
 * so a row's output bytes are the same for every M.  Asynchronous on `stream`. */
int qarl_harness_rmsnorm(qarl_ctx* ctx, const void* x_bf16, int64_t M, int64_t H, float eps,
                         void* out_bf16, void* stream);

/* Exercises the bounded-wait path every pipeline wait of the GEMM uses: one thread waits on an
 * mbarrier that nothing ever arrives on, with a limit of `limit_ns` nanoseconds (clamped to
 * [1 us, 100 ms]).  The wait gives up at the limit, records QARL_ERR_DEVICE_TIMEOUT in the
 * context's status word and the kernel returns normally: the context stays usable and
 * qarl_poll_device_status reports (and clears) the error.  Nothing traps, faults or hangs. */
int qarl_harness_wait_selftest(qarl_ctx* ctx, uint64_t limit_ns, void* stream);

/* The two calls below exist so that a test can watch the pipeline of the FP8 GEMMs and of the one-launch
 * router give up on a wait (the library never needs them).  Both only store a value in the context (host side, not
 * synchronized with calls running on other threads); it applies to the GEMM kernels launched
 * through `ctx` afterwards.
 *
 * qarl_harness_set_wait_limit_ns: the bound, in nanoseconds, of every barrier wait inside those
 * kernels (0 restores the default of 2 s; other values are clamped to [1 us, 2 s]).
 *
 * qarl_harness_stop_producer_after: the TMA producer of every CTA stops arming shared-memory
 * stages after `stages` of them (a negative value restores normal operation).  It waits for its
 * copies in flight and leaves its loop; nothing else is told.  The MMA role then waits on a stage
 * that nothing fills: its bounded wait runs out, it records QARL_ERR_DEVICE_TIMEOUT and raises the
 * CTA's abort flag; every other role leaves its loop at its next wait; the MMA role waits
 * (bounded) for the MMAs it had issued; TMEM is freed and the kernel returns.  Outputs of such a
 * call are unspecified; the context stays usable and qarl_poll_device_status reports the error.
 * Nothing traps, faults or spins without a bound. */
int qarl_harness_set_wait_limit_ns(qarl_ctx* ctx, uint64_t limit_ns);
int qarl_harness_stop_producer_after(qarl_ctx* ctx, int64_t stages);

/* The grouped FP8 GEMM has two kernels that produce the same bytes: the wide-tile one (128 token rows
 * x 256 weight rows per tile) and the swapped-operand one for decode-sized groups (128 weight rows x
 * at most 32 token rows); a decode-sized qarl_moe_fwd runs the latter once for the whole layer (gate_up
 * tiles, down tiles and the k-sum in one launch).  The library picks by size; this call forces one
 * (1 = wide, 2 = decode where it applies -- grouped calls with K <= 8192 --, one launch per projection
 * and a separate combine) or restores the automatic choice (0), so that a test can run one input
 * through each and compare.  A value other than 0 also makes qarl_router_fwd take its two-launch form.
 * Host side only, stored in the context. */
int qarl_harness_set_gemm_path(qarl_ctx* ctx, int path);

/* Roofline denominators measured with the library's own instructions (used by the benchmark; the
 * paper has no counterpart).  Both only launch a kernel on `stream`; the caller times it with
 * CUDA events.
 *
 * qarl_harness_fp8_mma_peak: every SM issues `kblocks_per_sm` back-to-back K-blocks of four
 * tcgen05.mma kind::f8f6f4 instructions (128 x 256 x 32, e4m3 operands resident in shared memory,
 * fp32 accumulators in TMEM) -- the instruction shape and operand path of the FP8 GEMM without its
 * loads, promotion and epilogue.  *flop_out (host pointer, may be NULL) receives the floating-point
 * operations the launch performs (2 * 128 * 256 * 128 per K-block per SM).
 *
 * qarl_harness_read_stream: reads `bytes` bytes (a multiple of 16, 16-byte aligned device pointer)
 * once with 16-byte loads, eight in flight per thread, and stores nothing (sink4: 4 writable device
 * bytes that are practically never written). */
int qarl_harness_fp8_mma_peak(qarl_ctx* ctx, int64_t kblocks_per_sm, double* flop_out, void* stream);
int qarl_harness_read_stream(qarl_ctx* ctx, const void* buf, size_t bytes, void* sink4, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* QARL_HARNESS_H_ */
