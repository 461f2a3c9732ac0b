"""Thin Python binding of the C-ABI library ``libqarl.so`` (see ``include/qarl.h``).

Argument marshalling only: every step of the quantized forward runs in the library's CUDA
kernels.  torch is used for device memory and streams.  There is no CPU path: loading fails
loudly if the library has not been built, and creating a context fails without an sm_100
device.
"""
from __future__ import annotations

import ctypes as C
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libqarl.so")

QARL_OK = 0
STATUS_NAMES = {
    0: "QARL_OK", -1: "QARL_ERR_INVALID_ARG", -2: "QARL_ERR_UNSUPPORTED_SHAPE",
    -3: "QARL_ERR_MISALIGNED", -4: "QARL_ERR_WORKSPACE_TOO_SMALL",
    -5: "QARL_ERR_UNSUPPORTED_DEVICE", -6: "QARL_ERR_CUDA", -7: "QARL_ERR_DEVICE_TIMEOUT",
    -8: "QARL_ERR_BAD_EXPERT_ID",
}

# every symbol include/qarl.h declares
EXPORTS = [
    "qarl_create", "qarl_destroy", "qarl_status_string", "qarl_poll_device_status",
    "qarl_last_cuda_error", "qarl_quantize_weight", "qarl_quantize_act",
    "qarl_linear_workspace_bytes", "qarl_linear_fwd", "qarl_linear_fwd_q",
    "qarl_moe_workspace_bytes", "qarl_moe_fwd", "qarl_launch_count",
    "qarl_profile_begin", "qarl_profile_end", "qarl_linear_fwd_static",
    "qarl_quantize_weight_w4", "qarl_linear_fwd_w4a16", "qarl_moe_w4a16_workspace_bytes",
    "qarl_moe_fwd_w4a16", "qarl_linear_bwd", "qarl_quantize_weight_publish",
    "qarl_tbpo_workspace_bytes", "qarl_tbpo_loss", "qarl_router_fwd", "qarl_grouped_linear_bwd", "qarl_moe_bwd_workspace_bytes", "qarl_moe_bwd",
    "qarl_moe_dispatch_workspace_bytes", "qarl_moe_dispatch", "qarl_moe_experts_workspace_bytes",
    "qarl_moe_experts_fwd", "qarl_moe_combine_sorted",
    "qarl_quantize_weight_w4_publish", "qarl_quantize_weight_fp4", "qarl_linear_fwd_fp4a16", "qarl_moe_fwd_fp4a16",
]
STATIC_LINEAR_MAX_ELEMS = 4 * 1024 * 1024
HARNESS_EXPORTS = ["qarl_harness_rmsnorm", "qarl_harness_wait_selftest", "qarl_harness_set_wait_limit_ns",
                   "qarl_harness_stop_producer_after", "qarl_harness_fp8_mma_peak", "qarl_harness_read_stream",
                   "qarl_harness_set_gemm_path"]
STAGES = ["quantize_weight", "quantize_act", "linear_gemm", "permute", "gate_up_gemm", "down_gemm",
          "combine", "bwd_dx", "bwd_dw", "tbpo", "router", "bwd_elementwise", "moe_decode_layer"]


class QarlError(RuntimeError):
    def __init__(self, status: int, detail: str = ""):
        self.status = status
        name = STATUS_NAMES.get(status, str(status))
        super().__init__(f"{name}{': ' + detail if detail else ''}")


class TbpoParams(C.Structure):
    _fields_ = [("eps_h", C.c_double), ("delta_l", C.c_double), ("delta_h", C.c_double), ("cap", C.c_double)]


class MoeDebug(C.Structure):
    _fields_ = [("expert_offsets", C.c_void_p), ("sorted_pair", C.c_void_p),
                ("gate_up_bf16", C.c_void_p), ("h_bf16", C.c_void_p), ("h_codes", C.c_void_p),
                ("h_scales", C.c_void_p), ("down_f32", C.c_void_p)]


_lib = None


def load() -> C.CDLL:
    """Load libqarl.so and declare its signatures.  Raises if the library is not built."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(
            f"{LIB_PATH} is missing: build it with `python -m paper_2604_07853_b200.build` "
            "(there is no CPU fallback)")
    L = C.CDLL(LIB_PATH)
    i64, p, sz = C.c_int64, C.c_void_p, C.c_size_t
    L.qarl_create.restype = C.c_int
    L.qarl_create.argtypes = [C.POINTER(p), C.c_int]
    L.qarl_destroy.restype = None
    L.qarl_destroy.argtypes = [p]
    L.qarl_status_string.restype = C.c_char_p
    L.qarl_status_string.argtypes = [C.c_int]
    L.qarl_poll_device_status.restype = C.c_int
    L.qarl_poll_device_status.argtypes = [p, p]
    L.qarl_last_cuda_error.restype = C.c_char_p
    L.qarl_last_cuda_error.argtypes = [p]
    L.qarl_quantize_weight.restype = C.c_int
    L.qarl_quantize_weight.argtypes = [p, p, i64, i64, i64, p, p, p]
    L.qarl_quantize_act.restype = C.c_int
    L.qarl_quantize_act.argtypes = [p, p, i64, i64, i64, p, p, p]
    L.qarl_linear_workspace_bytes.restype = sz
    L.qarl_linear_workspace_bytes.argtypes = [i64, i64, i64]
    L.qarl_linear_fwd.restype = C.c_int
    L.qarl_linear_fwd.argtypes = [p, p, i64, i64, p, p, i64, p, p, p, sz, p]
    L.qarl_linear_fwd_q.restype = C.c_int
    L.qarl_linear_fwd_q.argtypes = [p, p, p, i64, i64, p, p, i64, p, p, p]
    L.qarl_moe_workspace_bytes.restype = sz
    L.qarl_moe_workspace_bytes.argtypes = [i64, i64, i64, i64, i64]
    L.qarl_moe_fwd.restype = C.c_int
    L.qarl_moe_fwd.argtypes = [p, p, p, p, i64, i64, i64, i64, i64, p, p, p, p, p, p, sz,
                               C.POINTER(MoeDebug), p]
    L.qarl_launch_count.restype = i64
    L.qarl_launch_count.argtypes = [p]
    L.qarl_profile_begin.restype = C.c_int
    L.qarl_profile_begin.argtypes = [p, C.c_int]
    L.qarl_profile_end.restype = C.c_int
    L.qarl_profile_end.argtypes = [p, C.POINTER(C.c_double), C.POINTER(C.c_int64)]
    L.qarl_linear_fwd_static.restype = C.c_int
    L.qarl_linear_fwd_static.argtypes = [p, p, i64, i64, p, p, i64, p, p]
    L.qarl_quantize_weight_w4.restype = C.c_int
    L.qarl_quantize_weight_w4.argtypes = [p, p, i64, i64, i64, p, p, p, p]
    L.qarl_linear_fwd_w4a16.restype = C.c_int
    L.qarl_linear_fwd_w4a16.argtypes = [p, p, i64, i64, p, p, p, i64, p, p, p]
    L.qarl_moe_w4a16_workspace_bytes.restype = sz
    L.qarl_moe_w4a16_workspace_bytes.argtypes = [i64, i64, i64, i64, i64]
    L.qarl_moe_fwd_w4a16.restype = C.c_int
    L.qarl_moe_fwd_w4a16.argtypes = [p, p, p, p, i64, i64, i64, i64, i64, p, p, p, p, p, p, p, p, sz,
                                     C.POINTER(MoeDebug), p]
    L.qarl_quantize_weight_publish.restype = C.c_int
    L.qarl_quantize_weight_publish.argtypes = [p, p, i64, i64, i64, p, p, p, p, p]
    L.qarl_tbpo_workspace_bytes.restype = sz
    L.qarl_tbpo_workspace_bytes.argtypes = [i64, i64]
    L.qarl_tbpo_loss.restype = C.c_int
    L.qarl_tbpo_loss.argtypes = [p, p, p, p, p, p, i64, i64, C.POINTER(TbpoParams), p, p, p, p, p, p, p, sz, p]
    L.qarl_grouped_linear_bwd.restype = C.c_int
    L.qarl_grouped_linear_bwd.argtypes = [p, p, p, p, p, i64, i64, i64, i64, p, p, p, p]
    L.qarl_moe_bwd_workspace_bytes.restype = sz
    L.qarl_moe_bwd_workspace_bytes.argtypes = [i64, i64, i64, i64, i64]
    L.qarl_moe_bwd.restype = C.c_int
    L.qarl_moe_bwd.argtypes = [p, p, p, p, i64, i64, i64, i64, i64, p, p, p, p, p, p, p, p, p, p, p, sz, p]
    L.qarl_moe_dispatch_workspace_bytes.restype = sz
    L.qarl_moe_dispatch_workspace_bytes.argtypes = [i64, i64, i64]
    L.qarl_moe_dispatch.restype = C.c_int
    L.qarl_moe_dispatch.argtypes = [p, p, p, p, i64, i64, i64, i64, p, p, p, p, p, p, sz, p]
    L.qarl_moe_experts_workspace_bytes.restype = sz
    L.qarl_moe_experts_workspace_bytes.argtypes = [i64, i64]
    L.qarl_moe_experts_fwd.restype = C.c_int
    L.qarl_moe_experts_fwd.argtypes = [p, p, p, p, p, i64, i64, i64, i64, p, p, p, p, p, p, sz, p]
    L.qarl_moe_combine_sorted.restype = C.c_int
    L.qarl_moe_combine_sorted.argtypes = [p, p, p, p, i64, i64, i64, i64, p, p]
    L.qarl_quantize_weight_fp4.restype = C.c_int
    L.qarl_quantize_weight_fp4.argtypes = [p, p, i64, i64, i64, p, p, p, p, p]
    L.qarl_linear_fwd_fp4a16.restype = C.c_int
    L.qarl_linear_fwd_fp4a16.argtypes = [p, p, i64, i64, p, p, i64, p, p, p]
    L.qarl_moe_fwd_fp4a16.restype = C.c_int
    L.qarl_moe_fwd_fp4a16.argtypes = [p, p, p, p, i64, i64, i64, i64, i64, p, p, p, p, p, p, sz, p, p]
    L.qarl_quantize_weight_w4_publish.restype = C.c_int
    L.qarl_quantize_weight_w4_publish.argtypes = [p, p, i64, i64, i64, p, p, p, p, p, p, p]
    L.qarl_router_fwd.restype = C.c_int
    L.qarl_router_fwd.argtypes = [p, p, i64, i64, p, i64, i64, p, p, p, p]
    L.qarl_linear_bwd.restype = C.c_int
    L.qarl_linear_bwd.argtypes = [p, p, p, p, i64, i64, i64, p, p, p, p]
    L.qarl_harness_rmsnorm.restype = C.c_int
    L.qarl_harness_rmsnorm.argtypes = [p, p, i64, i64, C.c_float, p, p]
    L.qarl_harness_wait_selftest.restype = C.c_int
    L.qarl_harness_wait_selftest.argtypes = [p, C.c_uint64, p]
    L.qarl_harness_set_wait_limit_ns.restype = C.c_int
    L.qarl_harness_set_wait_limit_ns.argtypes = [p, C.c_uint64]
    L.qarl_harness_stop_producer_after.restype = C.c_int
    L.qarl_harness_stop_producer_after.argtypes = [p, i64]
    L.qarl_harness_set_gemm_path.restype = C.c_int
    L.qarl_harness_set_gemm_path.argtypes = [p, C.c_int]
    L.qarl_harness_fp8_mma_peak.restype = C.c_int
    L.qarl_harness_fp8_mma_peak.argtypes = [p, i64, C.POINTER(C.c_double), p]
    L.qarl_harness_read_stream.restype = C.c_int
    L.qarl_harness_read_stream.argtypes = [p, p, sz, p, p]
    _lib = L
    return L


def _ptr(t: torch.Tensor | None):
    return None if t is None else C.c_void_p(t.data_ptr())


def _stream():
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


class Context:
    """One qarl_ctx on one CUDA device.  Methods take and return torch CUDA tensors; bf16
    tensors are torch.bfloat16, codes torch.uint8, scales torch.float32."""

    def __init__(self, device: int = 0):
        self.lib = load()
        if not torch.cuda.is_available():
            raise QarlError(-5, "no CUDA device (the library has no CPU fallback)")
        self.device = torch.device("cuda", device)
        h = C.c_void_p()
        rc = self.lib.qarl_create(C.byref(h), device)
        if rc != QARL_OK:
            raise QarlError(rc)
        self.h = h
        self._ws: torch.Tensor | None = None

    def close(self):
        if getattr(self, "h", None):
            self.lib.qarl_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # ------------------------------------------------------------------ helpers
    def _check(self, rc: int):
        if rc != QARL_OK:
            detail = self.lib.qarl_last_cuda_error(self.h).decode() if rc == -6 else ""
            raise QarlError(rc, detail)

    def workspace(self, nbytes: int) -> torch.Tensor:
        """A cached device scratch buffer of at least nbytes (256-byte aligned)."""
        if self._ws is None or self._ws.numel() < nbytes:
            self._ws = torch.empty(max(nbytes, 256), dtype=torch.uint8, device=self.device)
        return self._ws

    def poll(self) -> int:
        """Synchronize the current stream; return and clear the device status word."""
        return int(self.lib.qarl_poll_device_status(self.h, _stream()))

    def check_device_status(self):
        rc = self.poll()
        if rc != QARL_OK:
            raise QarlError(rc)

    def launch_count(self) -> int:
        return int(self.lib.qarl_launch_count(self.h))

    def profile_begin(self, max_marks: int = 4096):
        """Start per-stage CUDA-event timing of this context's kernels."""
        self._check(self.lib.qarl_profile_begin(self.h, max_marks))

    def profile_end(self) -> dict:
        """Stop stage timing; returns {stage: (total_ms, launches)}."""
        n = len(STAGES)
        ms = (C.c_double * n)()
        cnt = (C.c_int64 * n)()
        self._check(self.lib.qarl_profile_end(self.h, ms, cnt))
        return {STAGES[i]: (float(ms[i]), int(cnt[i])) for i in range(n)}

    def harness_wait_selftest(self, limit_ns: int = 1_000_000):
        """Launch the bounded-wait self test (a wait nothing satisfies); poll() then returns -7."""
        self._check(self.lib.qarl_harness_wait_selftest(self.h, limit_ns, _stream()))

    def harness_set_wait_limit_ns(self, limit_ns: int):
        """Bound of every barrier wait in the GEMM kernels launched from now on (0: default)."""
        self._check(self.lib.qarl_harness_set_wait_limit_ns(self.h, limit_ns))

    def harness_stop_producer_after(self, stages: int):
        """FP8 GEMM TMA producers stop arming stages after `stages` (negative: normal operation)."""
        self._check(self.lib.qarl_harness_stop_producer_after(self.h, stages))

    def harness_set_gemm_path(self, path: int):
        """0: automatic choice of the grouped FP8 GEMM kernel, 1: wide tiles, 2: decode (swapped operands)."""
        self._check(self.lib.qarl_harness_set_gemm_path(self.h, path))

    def harness_fp8_mma_peak(self, kblocks_per_sm: int) -> float:
        """Launch the dense FP8 MMA peak kernel; returns the floating-point operations it performs."""
        fl = C.c_double(0.0)
        self._check(self.lib.qarl_harness_fp8_mma_peak(self.h, kblocks_per_sm, C.byref(fl), _stream()))
        return fl.value

    def harness_read_stream(self, buf: torch.Tensor, sink: torch.Tensor):
        """Launch the read-only streaming kernel over `buf` (bytes a multiple of 16)."""
        self._check(self.lib.qarl_harness_read_stream(self.h, _ptr(buf), buf.numel() * buf.element_size(),
                                                      _ptr(sink), _stream()))

    def harness_rmsnorm(self, x: torch.Tensor, eps: float = 1e-6, out=None):
        """Row-invariant RMSNorm (weight 1) used by the alignment-stack test; not part of the API."""
        assert x.dtype == torch.bfloat16 and x.is_contiguous()
        M, H = x.shape
        y = out if out is not None else torch.empty_like(x)
        self._check(self.lib.qarl_harness_rmsnorm(self.h, _ptr(x), M, H, eps, _ptr(y), _stream()))
        return y

    # ------------------------------------------------------------------ calls
    def quantize_weight(self, w: torch.Tensor, codes=None, scales=None):
        """w bf16 [E, N, K] or [N, K] -> (codes u8 same shape, scales f32 [.., N/128, K/128])."""
        assert w.dtype == torch.bfloat16 and w.is_cuda and w.is_contiguous()
        shape = w.shape
        E, N, K = (1, *shape) if w.dim() == 2 else shape
        if codes is None:
            codes = torch.empty(shape, dtype=torch.uint8, device=w.device)
        if scales is None:
            scales = torch.empty((*shape[:-2], N // 128, K // 128), dtype=torch.float32, device=w.device)
        self._check(self.lib.qarl_quantize_weight(self.h, _ptr(w), E, N, K, _ptr(codes), _ptr(scales), _stream()))
        return codes, scales

    def quantize_act(self, x: torch.Tensor, codes=None, scales=None):
        """x bf16 [M, K] (rows may be strided) -> (codes u8 [M, K], scales f32 [M, K/128])."""
        assert x.dtype == torch.bfloat16 and x.is_cuda and x.dim() == 2 and x.stride(1) == 1
        M, K = x.shape
        ldx = x.stride(0) if M > 1 else K
        if codes is None:
            codes = torch.empty((M, K), dtype=torch.uint8, device=x.device)
        if scales is None:
            scales = torch.empty((M, K // 128), dtype=torch.float32, device=x.device)
        self._check(self.lib.qarl_quantize_act(self.h, _ptr(x), M, K, ldx, _ptr(codes), _ptr(scales), _stream()))
        return codes, scales

    def linear_fwd(self, x, w_codes, w_scales, out=None, want_f32: bool = False):
        """y = blockscaled(quantize_act(x), W) -> y bf16 [M, N] (and the fp32 accumulator)."""
        assert x.dtype == torch.bfloat16 and x.is_contiguous()
        M, K = x.shape
        N = w_codes.shape[0]
        y = out if out is not None else torch.empty((M, N), dtype=torch.bfloat16, device=x.device)
        y32 = torch.empty((M, N), dtype=torch.float32, device=x.device) if want_f32 else None
        nbytes = int(self.lib.qarl_linear_workspace_bytes(M, N, K))
        ws = self.workspace(nbytes)
        self._check(self.lib.qarl_linear_fwd(self.h, _ptr(x), M, K, _ptr(w_codes), _ptr(w_scales), N,
                                             _ptr(y), _ptr(y32), _ptr(ws), ws.numel(), _stream()))
        return (y, y32) if want_f32 else y

    def linear_fwd_static(self, x, w_codes, w_scales, out):
        """qarl_linear_fwd_static: the dense projection for callers that cannot allocate device
        memory.  The scratch is a fixed array inside the library (M*K <= STATIC_LINEAR_MAX_ELEMS);
        the caller passes the input and a preallocated output, and this wrapper allocates
        nothing either.  Calls that overlap on the GPU race on that array."""
        assert x.dtype == torch.bfloat16 and x.is_contiguous() and out.dtype == torch.bfloat16
        M, K = x.shape
        N = w_codes.shape[0]
        assert out.shape == (M, N) and out.is_contiguous()
        rc = self.lib.qarl_linear_fwd_static(self.h, _ptr(x), M, K, _ptr(w_codes), _ptr(w_scales), N,
                                             _ptr(out), _stream())
        if rc != QARL_OK:
            raise QarlError(rc, self.lib.qarl_last_cuda_error(self.h).decode())
        return out

    def linear_fwd_q(self, x_codes, x_scales, w_codes, w_scales, out=None, want_f32: bool = False):
        M, K = x_codes.shape
        N = w_codes.shape[0]
        y = out if out is not None else torch.empty((M, N), dtype=torch.bfloat16, device=x_codes.device)
        y32 = torch.empty((M, N), dtype=torch.float32, device=x_codes.device) if want_f32 else None
        self._check(self.lib.qarl_linear_fwd_q(self.h, _ptr(x_codes), _ptr(x_scales), M, K, _ptr(w_codes),
                                               _ptr(w_scales), N, _ptr(y), _ptr(y32), _stream()))
        return (y, y32) if want_f32 else y

    def moe_workspace_bytes(self, M, H, I, E, k) -> int:
        return int(self.lib.qarl_moe_workspace_bytes(M, H, I, E, k))

    def moe_fwd(self, x, topk_ids, topk_weights, w13_codes, w13_scales, w2_codes, w2_scales,
                out=None, debug: bool = False, workspace: torch.Tensor | None = None, save=None):
        """One routed-expert FFN layer -> out bf16 [M, H] (and a dict of dumps if debug).
        save: dict(gate_up=bf16 [P, 2I], h=bf16 [P, I]) of caller-owned tensors that receive the
        activations the backward needs (expert-sorted order), without the other dumps."""
        assert x.dtype == torch.bfloat16 and x.is_contiguous()
        assert topk_ids.dtype == torch.int32 and topk_weights.dtype == torch.float32
        M, H = x.shape
        k = topk_ids.shape[1]
        E, I2, _ = w13_codes.shape
        I = I2 // 2
        P = M * k
        y = out if out is not None else torch.empty((M, H), dtype=torch.bfloat16, device=x.device)
        nbytes = self.moe_workspace_bytes(M, H, I, E, k)
        ws = workspace if workspace is not None else self.workspace(nbytes)
        d, dbg = None, None
        if save is not None:
            dbg = MoeDebug(None, None, save["gate_up"].data_ptr(), save["h"].data_ptr(), None, None, None)
        if debug:
            dev = x.device
            d = dict(expert_offsets=torch.zeros(E + 1, dtype=torch.int32, device=dev),
                     sorted_pair=torch.zeros(P, dtype=torch.int32, device=dev),
                     gate_up=torch.zeros((P, 2 * I), dtype=torch.bfloat16, device=dev),
                     h=torch.zeros((P, I), dtype=torch.bfloat16, device=dev),
                     h_codes=torch.zeros((P, I), dtype=torch.uint8, device=dev),
                     h_scales=torch.zeros((P, I // 128), dtype=torch.float32, device=dev),
                     down_f32=torch.zeros((P, H), dtype=torch.float32, device=dev))
            dbg = MoeDebug(d["expert_offsets"].data_ptr(), d["sorted_pair"].data_ptr(),
                           d["gate_up"].data_ptr(), d["h"].data_ptr(), d["h_codes"].data_ptr(),
                           d["h_scales"].data_ptr(), d["down_f32"].data_ptr())
        self._check(self.lib.qarl_moe_fwd(self.h, _ptr(x), _ptr(topk_ids), _ptr(topk_weights), M, H, I, E, k,
                                          _ptr(w13_codes), _ptr(w13_scales), _ptr(w2_codes), _ptr(w2_scales),
                                          _ptr(y), _ptr(ws), ws.numel(),
                                          C.byref(dbg) if dbg is not None else None, _stream()))
        return (y, d) if debug else y

    # ------------------------------------------------------------------ expert-parallel stages
    def moe_dispatch(self, x, topk_ids, topk_weights, E: int):
        """Quantize the tokens once and lay their (token, expert) rows out sorted by expert id ->
        dict(codes [P, H] u8, scales [P, H/128] f32, weights [P] f32, offsets [E+1] i32, pos_of_pair [P] i32)."""
        assert x.dtype == torch.bfloat16 and x.is_contiguous()
        assert topk_ids.dtype == torch.int32 and topk_weights.dtype == torch.float32
        M, H = x.shape
        k = topk_ids.shape[1]
        P, dev = M * k, x.device
        d = dict(codes=torch.empty((P, H), dtype=torch.uint8, device=dev),
                 scales=torch.empty((P, H // 128), dtype=torch.float32, device=dev),
                 weights=torch.empty(P, dtype=torch.float32, device=dev),
                 offsets=torch.empty(E + 1, dtype=torch.int32, device=dev),
                 pos_of_pair=torch.empty(P, dtype=torch.int32, device=dev))
        ws = self.workspace(int(self.lib.qarl_moe_dispatch_workspace_bytes(M, E, k)))
        self._check(self.lib.qarl_moe_dispatch(self.h, _ptr(x), _ptr(topk_ids), _ptr(topk_weights), M, H, E, k,
                                               _ptr(d["codes"]), _ptr(d["scales"]), _ptr(d["weights"]),
                                               _ptr(d["offsets"]), _ptr(d["pos_of_pair"]), _ptr(ws), ws.numel(),
                                               _stream()))
        return d

    def moe_experts_fwd(self, codes, scales, row_weights, offsets, w13_codes, w13_scales, w2_codes, w2_scales,
                        out=None):
        """gate_up, SwiGLU, down and the pair weight for rows grouped by local expert -> contrib bf16 [R, H]."""
        R, H = codes.shape
        E_local, I2, _ = w13_codes.shape
        I = I2 // 2
        assert offsets.dtype == torch.int32 and offsets.numel() == E_local + 1
        assert codes.is_contiguous() and scales.is_contiguous() and row_weights.is_contiguous()
        contrib = out if out is not None else torch.empty((R, H), dtype=torch.bfloat16, device=codes.device)
        assert contrib.is_contiguous() and contrib.dtype == torch.bfloat16
        ws = self.workspace(int(self.lib.qarl_moe_experts_workspace_bytes(R, I)))
        self._check(self.lib.qarl_moe_experts_fwd(self.h, _ptr(codes), _ptr(scales), _ptr(row_weights), _ptr(offsets),
                                                  R, H, I, E_local, _ptr(w13_codes), _ptr(w13_scales), _ptr(w2_codes),
                                                  _ptr(w2_scales), _ptr(contrib), _ptr(ws), ws.numel(), _stream()))
        return contrib

    def moe_combine_sorted(self, contrib_sorted, topk_ids, pos_of_pair, E: int):
        """The k-sum in ascending expert id over contributions held in dispatch order -> out bf16 [M, H]."""
        M, k = topk_ids.shape
        H = contrib_sorted.shape[1]
        out = torch.empty((M, H), dtype=torch.bfloat16, device=contrib_sorted.device)
        self._check(self.lib.qarl_moe_combine_sorted(self.h, _ptr(contrib_sorted), _ptr(topk_ids), _ptr(pos_of_pair),
                                                     M, H, E, k, _ptr(out), _stream()))
        return out

    # ------------------------------------------------------------------ W4A16
    def quantize_weight_w4(self, w: torch.Tensor, out=None):
        """w bf16 [E, N, K] or [N, K] -> (packed u8 [.., N, K/2], scales bf16 [.., K/128, N],
        zeros u8 [.., K/128, N]) in the library's storage order (see include/qarl.h).
        out: an earlier result of this call to overwrite."""
        assert w.dtype == torch.bfloat16 and w.is_cuda and w.is_contiguous()
        shape = w.shape
        E, N, K = (1, *shape) if w.dim() == 2 else shape
        if out is not None:
            packed, scales, zeros = out
        else:
            packed = torch.empty((*shape[:-1], K // 2), dtype=torch.uint8, device=w.device)
            scales = torch.empty((*shape[:-2], K // 128, N), dtype=torch.bfloat16, device=w.device)
            zeros = torch.empty((*shape[:-2], K // 128, N), dtype=torch.uint8, device=w.device)
        self._check(self.lib.qarl_quantize_weight_w4(self.h, _ptr(w), E, N, K, _ptr(packed), _ptr(scales),
                                                     _ptr(zeros), _stream()))
        return packed, scales, zeros

    def quantize_weight_w4_publish(self, w, out, pub):
        """quantize_weight_w4 writing a second, published copy (packed, scales, zeros) in the same launch."""
        assert w.dtype == torch.bfloat16 and w.is_cuda and w.is_contiguous()
        E, N, K = (1, *w.shape) if w.dim() == 2 else w.shape
        self._check(self.lib.qarl_quantize_weight_w4_publish(self.h, _ptr(w), E, N, K, _ptr(out[0]), _ptr(out[1]),
                                                             _ptr(out[2]), _ptr(pub[0]), _ptr(pub[1]), _ptr(pub[2]),
                                                             _stream()))
        return out

    def linear_fwd_w4a16(self, x, w_packed, w_scales, w_zeros, out=None, want_f32: bool = False):
        """y = x . w^T with 4-bit weights -> y bf16 [M, N] (and the fp32 accumulator if want_f32)."""
        assert x.dtype == torch.bfloat16 and x.is_contiguous()
        M, K = x.shape
        N = w_packed.shape[-2]
        y = out if out is not None else torch.empty((M, N), dtype=torch.bfloat16, device=x.device)
        y32 = torch.empty((M, N), dtype=torch.float32, device=x.device) if want_f32 else None
        self._check(self.lib.qarl_linear_fwd_w4a16(self.h, _ptr(x), M, K, _ptr(w_packed), _ptr(w_scales),
                                                   _ptr(w_zeros), N, _ptr(y), _ptr(y32), _stream()))
        return (y, y32) if want_f32 else y

    def moe_w4a16_workspace_bytes(self, M, H, I, E, k) -> int:
        return int(self.lib.qarl_moe_w4a16_workspace_bytes(M, H, I, E, k))

    def moe_fwd_w4a16(self, x, topk_ids, topk_weights, w13, w2, out=None, debug: bool = False,
                      workspace: torch.Tensor | None = None):
        """One routed-expert FFN layer on W4A16 weights; w13 and w2 are (packed, scales, zeros)."""
        assert x.dtype == torch.bfloat16 and x.is_contiguous()
        assert topk_ids.dtype == torch.int32 and topk_weights.dtype == torch.float32
        M, H = x.shape
        k = topk_ids.shape[1]
        E, I2, _ = w13[0].shape
        I = I2 // 2
        P = M * k
        y = out if out is not None else torch.empty((M, H), dtype=torch.bfloat16, device=x.device)
        ws = workspace if workspace is not None else self.workspace(self.moe_w4a16_workspace_bytes(M, H, I, E, k))
        d, dbg = None, None
        if debug:
            dev = x.device
            d = dict(expert_offsets=torch.zeros(E + 1, dtype=torch.int32, device=dev),
                     sorted_pair=torch.zeros(P, dtype=torch.int32, device=dev),
                     gate_up=torch.zeros((P, 2 * I), dtype=torch.bfloat16, device=dev),
                     h=torch.zeros((P, I), dtype=torch.bfloat16, device=dev),
                     down_f32=torch.zeros((P, H), dtype=torch.float32, device=dev))
            dbg = MoeDebug(d["expert_offsets"].data_ptr(), d["sorted_pair"].data_ptr(),
                           d["gate_up"].data_ptr(), d["h"].data_ptr(), None, None, d["down_f32"].data_ptr())
        self._check(self.lib.qarl_moe_fwd_w4a16(self.h, _ptr(x), _ptr(topk_ids), _ptr(topk_weights), M, H, I, E, k,
                                                _ptr(w13[0]), _ptr(w13[1]), _ptr(w13[2]),
                                                _ptr(w2[0]), _ptr(w2[1]), _ptr(w2[2]),
                                                _ptr(y), _ptr(ws), ws.numel(),
                                                C.byref(dbg) if dbg is not None else None, _stream()))
        return (y, d) if debug else y

    # ------------------------------------------------------------------ FP4A16 (e2m1 weights)
    def quantize_weight_fp4(self, w: torch.Tensor, out=None, pub=None):
        """w bf16 [E, N, K] or [N, K] -> (packed u8 [.., N, K/2], scales bf16 [.., K/128, N]) of e2m1 codes in
        the library's storage order.  out: an earlier result to overwrite; pub: a second (packed, scales)
        destination written in the same launch."""
        assert w.dtype == torch.bfloat16 and w.is_cuda and w.is_contiguous()
        shape = w.shape
        E, N, K = (1, *shape) if w.dim() == 2 else shape
        if out is not None:
            packed, scales = out
        else:
            packed = torch.empty((*shape[:-1], K // 2), dtype=torch.uint8, device=w.device)
            scales = torch.empty((*shape[:-2], K // 128, N), dtype=torch.bfloat16, device=w.device)
        pp, ps = pub if pub is not None else (None, None)
        self._check(self.lib.qarl_quantize_weight_fp4(self.h, _ptr(w), E, N, K, _ptr(packed), _ptr(scales),
                                                      _ptr(pp), _ptr(ps), _stream()))
        return packed, scales

    def linear_fwd_fp4a16(self, x, w_packed, w_scales, out=None, want_f32: bool = False):
        """y = x . w^T with e2m1 weights -> y bf16 [M, N] (and the fp32 accumulator if want_f32)."""
        assert x.dtype == torch.bfloat16 and x.is_contiguous()
        M, K = x.shape
        N = w_packed.shape[-2]
        y = out if out is not None else torch.empty((M, N), dtype=torch.bfloat16, device=x.device)
        y32 = torch.empty((M, N), dtype=torch.float32, device=x.device) if want_f32 else None
        self._check(self.lib.qarl_linear_fwd_fp4a16(self.h, _ptr(x), M, K, _ptr(w_packed), _ptr(w_scales), N,
                                                    _ptr(y), _ptr(y32), _stream()))
        return (y, y32) if want_f32 else y

    def moe_fwd_fp4a16(self, x, topk_ids, topk_weights, w13, w2, out=None, debug: bool = False,
                       workspace: torch.Tensor | None = None):
        """One routed-expert FFN layer on e2m1 weights; w13 and w2 are (packed, scales)."""
        assert x.dtype == torch.bfloat16 and x.is_contiguous()
        assert topk_ids.dtype == torch.int32 and topk_weights.dtype == torch.float32
        M, H = x.shape
        k = topk_ids.shape[1]
        E, I2, _ = w13[0].shape
        I = I2 // 2
        P = M * k
        y = out if out is not None else torch.empty((M, H), dtype=torch.bfloat16, device=x.device)
        ws = workspace if workspace is not None else self.workspace(self.moe_w4a16_workspace_bytes(M, H, I, E, k))
        d, dbg = None, None
        if debug:
            dev = x.device
            d = dict(expert_offsets=torch.zeros(E + 1, dtype=torch.int32, device=dev),
                     sorted_pair=torch.zeros(P, dtype=torch.int32, device=dev),
                     gate_up=torch.zeros((P, 2 * I), dtype=torch.bfloat16, device=dev),
                     h=torch.zeros((P, I), dtype=torch.bfloat16, device=dev),
                     down_f32=torch.zeros((P, H), dtype=torch.float32, device=dev))
            dbg = MoeDebug(d["expert_offsets"].data_ptr(), d["sorted_pair"].data_ptr(),
                           d["gate_up"].data_ptr(), d["h"].data_ptr(), None, None, d["down_f32"].data_ptr())
        self._check(self.lib.qarl_moe_fwd_fp4a16(self.h, _ptr(x), _ptr(topk_ids), _ptr(topk_weights), M, H, I, E, k,
                                                 _ptr(w13[0]), _ptr(w13[1]), _ptr(w2[0]), _ptr(w2[1]),
                                                 _ptr(y), _ptr(ws), ws.numel(),
                                                 C.byref(dbg) if dbg is not None else None, _stream()))
        return (y, d) if debug else y

    def quantize_weight_publish(self, w, codes, scales, pub_codes, pub_scales):
        """quantize_weight writing a second, published copy of codes and scales in the same launch."""
        assert w.dtype == torch.bfloat16 and w.is_cuda and w.is_contiguous()
        E, N, K = (1, *w.shape) if w.dim() == 2 else w.shape
        self._check(self.lib.qarl_quantize_weight_publish(self.h, _ptr(w), E, N, K, _ptr(codes), _ptr(scales),
                                                          _ptr(pub_codes), _ptr(pub_scales), _stream()))
        return codes, scales

    # ------------------------------------------------------------------ backward
    def linear_bwd(self, dy, x, w, want_dx_f32: bool = False, dx: bool = True, dw: bool = True):
        """Straight-through backward of y = x . W^T on the bf16 masters ->
        (dX bf16 [M, K] or None, dX fp32 or None, dW fp32 [N, K] or None)."""
        for t in (dy, x, w):
            assert t.dtype == torch.bfloat16 and t.is_cuda and t.is_contiguous()
        M, N = dy.shape
        K = x.shape[1]
        assert x.shape == (M, K) and w.shape == (N, K)
        dxo = torch.empty((M, K), dtype=torch.bfloat16, device=dy.device) if dx else None
        dx32 = torch.empty((M, K), dtype=torch.float32, device=dy.device) if (dx and want_dx_f32) else None
        dwo = torch.empty((N, K), dtype=torch.float32, device=dy.device) if dw else None
        self._check(self.lib.qarl_linear_bwd(self.h, _ptr(dy), _ptr(x), _ptr(w), M, N, K, _ptr(dxo), _ptr(dx32),
                                             _ptr(dwo), _stream()))
        return dxo, dx32, dwo

    def grouped_linear_bwd(self, dy, x, w, offsets, want_dx_f32: bool = False, dx: bool = True, dw: bool = True):
        """Backward of an expert projection on expert-sorted rows: dy [P, N], x [P, K], w [E, N, K] bf16,
        offsets i32 [E+1] -> (dX bf16 [P, K] or None, dX fp32 or None, dW fp32 [E, N, K] or None)."""
        for t in (dy, x, w):
            assert t.dtype == torch.bfloat16 and t.is_cuda and t.is_contiguous()
        assert offsets.dtype == torch.int32 and offsets.is_cuda
        P, N = dy.shape
        E, _, K = w.shape
        dxo = torch.empty((P, K), dtype=torch.bfloat16, device=w.device) if dx else None
        dx32 = torch.empty((P, K), dtype=torch.float32, device=w.device) if (dx and want_dx_f32) else None
        dwo = torch.empty((E, N, K), dtype=torch.float32, device=w.device) if dw else None
        self._check(self.lib.qarl_grouped_linear_bwd(self.h, _ptr(dy), _ptr(x), _ptr(w), _ptr(offsets), P, N, K, E,
                                                     _ptr(dxo), _ptr(dx32), _ptr(dwo), _stream()))
        return dxo, dx32, dwo

    def moe_bwd(self, x, topk_ids, topk_weights, w13, w2, gate_up, h, dout, down_f32=None, out=None, workspace=None):
        """Backward of the routed-expert FFN layer on bf16 masters w13 [E, 2I, H], w2 [E, H, I] and the
        forward's saved bf16 gate_up [P, 2I] / h [P, I] (expert-sorted) ->
        dict(dx bf16 [M, H], dw13 f32, dw2 f32, dwts f32 [M, k] or None)."""
        M, H = x.shape
        k = topk_ids.shape[1]
        E, I2, _ = w13.shape
        I = I2 // 2
        dev = x.device
        if out is None:
            out = dict(dx=torch.empty((M, H), dtype=torch.bfloat16, device=dev),
                       dw13=torch.empty((E, 2 * I, H), dtype=torch.float32, device=dev),
                       dw2=torch.empty((E, H, I), dtype=torch.float32, device=dev),
                       dwts=torch.empty((M, k), dtype=torch.float32, device=dev) if down_f32 is not None else None)
        ws = workspace if workspace is not None else self.workspace(max(int(self.lib.qarl_moe_bwd_workspace_bytes(M, H, I, E, k)), 256))
        self._check(self.lib.qarl_moe_bwd(self.h, _ptr(x), _ptr(topk_ids), _ptr(topk_weights), M, H, I, E, k, _ptr(w13),
                                          _ptr(w2), _ptr(gate_up), _ptr(h), _ptr(dout), _ptr(down_f32), _ptr(out["dx"]),
                                          _ptr(out["dw13"]), _ptr(out["dw2"]), _ptr(out["dwts"]), _ptr(ws), ws.numel(),
                                          _stream()))
        return out

    # ------------------------------------------------------------------ TBPO
    def tbpo_loss(self, lp_cur, lp_old_learner, lp_old_sampler, offsets, adv, eps_h=4e-4, delta_l=3e-4,
                  delta_h=7e-4, cap=2.0, want_grad: bool = True, out=None, workspace=None):
        """Sequence-level TBPO surrogate over B packed responses -> dict(r, w, J f64 [B], flags i32 [B],
        grad f32 [T] or None, loss f64 [1]) of device tensors.  out: an earlier result to overwrite."""
        for t in (lp_cur, lp_old_learner, lp_old_sampler, adv):
            assert t.dtype == torch.float32 and t.is_cuda and t.is_contiguous()
        assert offsets.dtype == torch.int64 and offsets.is_cuda
        B, T = adv.shape[0], lp_cur.shape[0]
        dev = lp_cur.device
        if out is None:
            out = dict(r=torch.empty(B, dtype=torch.float64, device=dev), w=torch.empty(B, dtype=torch.float64, device=dev),
                       J=torch.empty(B, dtype=torch.float64, device=dev), flags=torch.empty(B, dtype=torch.int32, device=dev),
                       grad=torch.empty(T, dtype=torch.float32, device=dev) if want_grad else None,
                       loss=torch.empty(1, dtype=torch.float64, device=dev))
        ws = workspace if workspace is not None else self.workspace(max(int(self.lib.qarl_tbpo_workspace_bytes(B, T)), 256))
        prm = TbpoParams(eps_h, delta_l, delta_h, cap)
        self._check(self.lib.qarl_tbpo_loss(self.h, _ptr(lp_cur), _ptr(lp_old_learner), _ptr(lp_old_sampler),
                                            _ptr(offsets), _ptr(adv), B, T, C.byref(prm), _ptr(out["r"]), _ptr(out["w"]),
                                            _ptr(out["J"]), _ptr(out["flags"]), _ptr(out["grad"]), _ptr(out["loss"]),
                                            _ptr(ws), ws.numel(), _stream()))
        return out

    # ------------------------------------------------------------------ router
    def router_fwd(self, x, w_router, k: int):
        """x bf16 [M, H], w_router bf16 [E, H] -> (logits f32 [M, E], ids i32 [M, k], weights f32 [M, k])."""
        assert x.dtype == torch.bfloat16 and w_router.dtype == torch.bfloat16 and x.is_contiguous() and w_router.is_contiguous()
        M, H = x.shape
        E = w_router.shape[0]
        logits = torch.empty((M, E), dtype=torch.float32, device=x.device)
        ids = torch.empty((M, k), dtype=torch.int32, device=x.device)
        wts = torch.empty((M, k), dtype=torch.float32, device=x.device)
        self._check(self.lib.qarl_router_fwd(self.h, _ptr(x), M, H, _ptr(w_router), E, k, _ptr(logits), _ptr(ids),
                                             _ptr(wts), _stream()))
        return logits, ids, wts
