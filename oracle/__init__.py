"""ctypes front end of the CPU oracle (``qarl_oracle.c``).

TEST INFRASTRUCTURE ONLY: importable from ``tests/``, the smoke check and the benchmark's
CPU-baseline leg.  The product path (the CUDA library and its Python binding) never imports
this package, and this package never imports the product path.

bf16 tensors travel as numpy ``uint16`` arrays of bit patterns.
"""
from __future__ import annotations

import ctypes as C

import numpy as np

from .build import build as _build

_lib = None


def lib() -> C.CDLL:
    global _lib
    if _lib is None:
        _lib = C.CDLL(_build())
        L = _lib
        i64, p = C.c_int64, C.c_void_p
        L.oracle_bf16_rne.restype = C.c_uint16
        L.oracle_bf16_rne.argtypes = [C.c_float]
        L.oracle_e4m3_decode.restype = C.c_double
        L.oracle_e4m3_decode.argtypes = [C.c_uint8]
        L.oracle_e4m3_encode.restype = C.c_uint8
        L.oracle_e4m3_encode.argtypes = [C.c_float]
        L.oracle_e4m3_encode_array.restype = None
        L.oracle_e4m3_encode_array.argtypes = [p, i64, p]
        L.oracle_bf16_rne_array.restype = None
        L.oracle_bf16_rne_array.argtypes = [p, i64, p]
        L.oracle_quantize_weight.restype = C.c_int
        L.oracle_quantize_weight.argtypes = [p, i64, i64, i64, p, p]
        L.oracle_quantize_act.restype = C.c_int
        L.oracle_quantize_act.argtypes = [p, i64, i64, i64, p, p]
        L.oracle_linear_q.restype = C.c_int
        L.oracle_linear_q.argtypes = [p, p, i64, i64, p, p, i64, p, p]
        L.oracle_linear.restype = C.c_int
        L.oracle_linear.argtypes = [p, i64, i64, p, p, i64, p, p]
        L.oracle_permute.restype = C.c_int
        L.oracle_permute.argtypes = [p, i64, i64, i64, p, p, p]
        L.oracle_swiglu.restype = None
        L.oracle_swiglu.argtypes = [p, i64, i64, p]
        L.oracle_combine.restype = None
        L.oracle_combine.argtypes = [p, p, p, i64, i64, i64, p]
        L.oracle_moe.restype = C.c_int
        L.oracle_moe.argtypes = [p, p, p, i64, i64, i64, i64, i64, p, p, p, p, p, p, p, p, p, p]
        L.oracle_quantize_weight_w4.restype = C.c_int
        L.oracle_quantize_weight_w4.argtypes = [p, i64, i64, i64, p, p, p]
        L.oracle_dequant_w4.restype = None
        L.oracle_dequant_w4.argtypes = [p, p, p, i64, i64, p]
        L.oracle_e2m1_decode.restype = C.c_double
        L.oracle_e2m1_decode.argtypes = [C.c_uint8]
        L.oracle_e2m1_encode.restype = C.c_uint8
        L.oracle_e2m1_encode.argtypes = [C.c_float]
        L.oracle_quantize_weight_fp4.restype = C.c_int
        L.oracle_quantize_weight_fp4.argtypes = [p, i64, i64, i64, p, p]
        L.oracle_dequant_fp4.restype = None
        L.oracle_dequant_fp4.argtypes = [p, p, i64, i64, p]
        L.oracle_linear_bf16.restype = None
        L.oracle_linear_bf16.argtypes = [p, i64, i64, p, i64, p, p]
        L.oracle_moe_w4a16.restype = C.c_int
        L.oracle_moe_w4a16.argtypes = [p, p, p, i64, i64, i64, i64, i64, p, p, p, p, p, p]
        L.oracle_linear_bwd.restype = None
        L.oracle_linear_bwd.argtypes = [p, p, p, i64, i64, i64, p, p, p]
        L.oracle_tbpo.restype = None
        L.oracle_tbpo.argtypes = [p, p, p, p, p, i64] + [C.c_double] * 4 + [p] * 6
        L.oracle_router_topk.restype = None
        L.oracle_router_topk.argtypes = [p, i64, i64, i64, p, p]
        L.oracle_swiglu_bwd.restype = None
        L.oracle_swiglu_bwd.argtypes = [p, p, i64, i64, p]
        L.oracle_num_threads.restype = C.c_int
        L.oracle_num_threads.argtypes = []
    return _lib


def _ptr(a: np.ndarray | None):
    if a is None:
        return None
    assert a.flags["C_CONTIGUOUS"]
    return a.ctypes.data_as(C.c_void_p)


def _c(a, dtype) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=dtype)


class OracleError(RuntimeError):
    def __init__(self, code: int):
        super().__init__(f"oracle returned status {code}")
        self.code = code


def num_threads() -> int:
    return int(lib().oracle_num_threads())


def e4m3_decode_table() -> np.ndarray:
    """All 256 code values as float64 (NaN at 0x7F / 0xFF)."""
    return np.array([lib().oracle_e4m3_decode(c) for c in range(256)], dtype=np.float64)


def e4m3_encode(v) -> np.ndarray:
    v = _c(v, np.float32)
    out = np.empty(v.shape, dtype=np.uint8)
    lib().oracle_e4m3_encode_array(_ptr(v), v.size, _ptr(out))
    return out


def bf16_rne(v) -> np.ndarray:
    v = _c(v, np.float32)
    out = np.empty(v.shape, dtype=np.uint16)
    lib().oracle_bf16_rne_array(_ptr(v), v.size, _ptr(out))
    return out


def quantize_weight(w_bits: np.ndarray) -> tuple[np.ndarray, np.ndarray]:
    """w bf16 bits [E, N, K] or [N, K] -> (codes u8 same shape, scales f32 [.., N/128, K/128])."""
    w = _c(w_bits, np.uint16)
    squeeze = w.ndim == 2
    if squeeze:
        w = w[None]
    E, N, K = w.shape
    codes = np.empty((E, N, K), dtype=np.uint8)
    scales = np.empty((E, N // 128, K // 128), dtype=np.float32)
    rc = lib().oracle_quantize_weight(_ptr(w), E, N, K, _ptr(codes), _ptr(scales))
    if rc:
        raise OracleError(rc)
    return (codes[0], scales[0]) if squeeze else (codes, scales)


def quantize_act(x_bits: np.ndarray) -> tuple[np.ndarray, np.ndarray]:
    """x bf16 bits [M, K] -> (codes u8 [M, K], scales f32 [M, K/128])."""
    x = _c(x_bits, np.uint16)
    M, K = x.shape
    codes = np.empty((M, K), dtype=np.uint8)
    scales = np.empty((M, K // 128), dtype=np.float32)
    rc = lib().oracle_quantize_act(_ptr(x), M, K, K, _ptr(codes), _ptr(scales))
    if rc:
        raise OracleError(rc)
    return codes, scales


def linear_q(xc, xs, wc, ws) -> tuple[np.ndarray, np.ndarray]:
    """Block-scaled linear from codes and scales -> (y fp32 [M, N], y bf16 bits [M, N])."""
    xc, xs, wc, ws = _c(xc, np.uint8), _c(xs, np.float32), _c(wc, np.uint8), _c(ws, np.float32)
    M, K = xc.shape
    N = wc.shape[0]
    assert wc.shape[1] == K
    y32 = np.empty((M, N), dtype=np.float32)
    y16 = np.empty((M, N), dtype=np.uint16)
    rc = lib().oracle_linear_q(_ptr(xc), _ptr(xs), M, K, _ptr(wc), _ptr(ws), N, _ptr(y32), _ptr(y16))
    if rc:
        raise OracleError(rc)
    return y32, y16


def linear(x_bits, wc, ws) -> tuple[np.ndarray, np.ndarray]:
    """y = blockscaled(quantize_act(x), W) -> (y fp32, y bf16 bits)."""
    x, wc, ws = _c(x_bits, np.uint16), _c(wc, np.uint8), _c(ws, np.float32)
    M, K = x.shape
    N = wc.shape[0]
    y32 = np.empty((M, N), dtype=np.float32)
    y16 = np.empty((M, N), dtype=np.uint16)
    rc = lib().oracle_linear(_ptr(x), M, K, _ptr(wc), _ptr(ws), N, _ptr(y32), _ptr(y16))
    if rc:
        raise OracleError(rc)
    return y32, y16


def permute(ids, E: int) -> tuple[np.ndarray, np.ndarray, np.ndarray]:
    """ids int32 [M, k] -> (offsets [E+1], sorted_pair [M*k], pos_of_pair [M*k])."""
    ids = _c(ids, np.int32)
    M, k = ids.shape
    offsets = np.empty(E + 1, dtype=np.int32)
    sorted_pair = np.empty(M * k, dtype=np.int32)
    pos = np.empty(M * k, dtype=np.int32)
    rc = lib().oracle_permute(_ptr(ids), M, k, E, _ptr(offsets), _ptr(sorted_pair), _ptr(pos))
    if rc:
        raise OracleError(rc)
    return offsets, sorted_pair, pos


def swiglu(gate_up_bits) -> np.ndarray:
    """gate_up bf16 bits [P, 2I] -> h bf16 bits [P, I]."""
    gu = _c(gate_up_bits, np.uint16)
    P, I2 = gu.shape
    h = np.empty((P, I2 // 2), dtype=np.uint16)
    lib().oracle_swiglu(_ptr(gu), P, I2 // 2, _ptr(h))
    return h


def combine(y32, ids, wts) -> np.ndarray:
    """y32 fp32 [M*k, H] by flat pair id, ids/wts [M, k] -> out bf16 bits [M, H]."""
    y32, ids, wts = _c(y32, np.float32), _c(ids, np.int32), _c(wts, np.float32)
    M, k = ids.shape
    H = y32.shape[1]
    out = np.empty((M, H), dtype=np.uint16)
    lib().oracle_combine(_ptr(y32), _ptr(ids), _ptr(wts), M, k, H, _ptr(out))
    return out


def moe(x_bits, ids, wts, w13c, w13s, w2c, w2s, dumps: bool = False):
    """One routed MoE FFN layer.  Returns out bf16 bits [M, H], or (out, dict of dumps)
    with gate_up [P,2I], h [P,I], h_codes [P,I], h_scales [P,I/128], y32 [P,H] by pair id."""
    x, ids, wts = _c(x_bits, np.uint16), _c(ids, np.int32), _c(wts, np.float32)
    w13c, w13s = _c(w13c, np.uint8), _c(w13s, np.float32)
    w2c, w2s = _c(w2c, np.uint8), _c(w2s, np.float32)
    M, H = x.shape
    k = ids.shape[1]
    E, I2, _ = w13c.shape
    I = I2 // 2
    P = M * k
    out = np.empty((M, H), dtype=np.uint16)
    d = {}
    if dumps:
        d = dict(gate_up=np.empty((P, 2 * I), np.uint16), h=np.empty((P, I), np.uint16),
                 h_codes=np.empty((P, I), np.uint8), h_scales=np.empty((P, I // 128), np.float32),
                 y32=np.empty((P, H), np.float32))
    rc = lib().oracle_moe(_ptr(x), _ptr(ids), _ptr(wts), M, H, I, E, k,
                          _ptr(w13c), _ptr(w13s), _ptr(w2c), _ptr(w2s), _ptr(out),
                          _ptr(d.get("gate_up")), _ptr(d.get("h")), _ptr(d.get("h_codes")),
                          _ptr(d.get("h_scales")), _ptr(d.get("y32")))
    if rc:
        raise OracleError(rc)
    return (out, d) if dumps else out


# ---------------------------------------------------------------------------- W4A16
def quantize_weight_w4(w_bits: np.ndarray):
    """w bf16 bits [E, N, K] or [N, K] -> (packed u8 [.., N, K/2], scales f32 [.., N, K/128],
    zeros u8 [.., N, K/128]); unsigned 4-bit codes, one (s, z) per 128 K-elements of a row."""
    w = _c(w_bits, np.uint16)
    squeeze = w.ndim == 2
    if squeeze:
        w = w[None]
    E, N, K = w.shape
    packed = np.empty((E, N, K // 2), dtype=np.uint8)
    scales = np.empty((E, N, K // 128), dtype=np.float32)
    zeros = np.empty((E, N, K // 128), dtype=np.uint8)
    rc = lib().oracle_quantize_weight_w4(_ptr(w), E, N, K, _ptr(packed), _ptr(scales), _ptr(zeros))
    if rc:
        raise OracleError(rc)
    return (packed[0], scales[0], zeros[0]) if squeeze else (packed, scales, zeros)


def dequant_w4(packed, scales, zeros) -> np.ndarray:
    """-> w^ bf16 bits, same leading shape, last dim K."""
    packed, scales, zeros = _c(packed, np.uint8), _c(scales, np.float32), _c(zeros, np.uint8)
    K = packed.shape[-1] * 2
    rows = int(np.prod(packed.shape[:-1]))
    out = np.empty((*packed.shape[:-1], K), dtype=np.uint16)
    lib().oracle_dequant_w4(_ptr(packed), _ptr(scales), _ptr(zeros), rows, K, _ptr(out))
    return out


def e2m1_table() -> np.ndarray:
    """The 16 e2m1 code values (code 8 is -0)."""
    return np.array([lib().oracle_e2m1_decode(c) for c in range(16)], dtype=np.float64)


def e2m1_encode(values) -> np.ndarray:
    v = np.ascontiguousarray(values, dtype=np.float32)
    return np.array([lib().oracle_e2m1_encode(float(t)) for t in v.ravel()], dtype=np.uint8).reshape(v.shape)


def quantize_weight_fp4(w_bits: np.ndarray):
    """w bf16 bits [E, N, K] or [N, K] -> (packed u8 [.., N, K/2], scales f32 [.., N, K/128]);
    e2m1 codes, one scale per 128 K-elements of a row."""
    w = _c(w_bits, np.uint16)
    squeeze = w.ndim == 2
    if squeeze:
        w = w[None]
    E, N, K = w.shape
    packed = np.empty((E, N, K // 2), dtype=np.uint8)
    scales = np.empty((E, N, K // 128), dtype=np.float32)
    rc = lib().oracle_quantize_weight_fp4(_ptr(w), E, N, K, _ptr(packed), _ptr(scales))
    if rc:
        raise OracleError(rc)
    return (packed[0], scales[0]) if squeeze else (packed, scales)


def dequant_fp4(packed, scales) -> np.ndarray:
    """-> w^ bf16 bits, same leading shape, last dim K."""
    packed, scales = _c(packed, np.uint8), _c(scales, np.float32)
    K = packed.shape[-1] * 2
    rows = int(np.prod(packed.shape[:-1]))
    out = np.empty((*packed.shape[:-1], K), dtype=np.uint16)
    lib().oracle_dequant_fp4(_ptr(packed), _ptr(scales), rows, K, _ptr(out))
    return out


def linear_bf16(x_bits, w_hat_bits):
    """y = x . w^T on bf16 operands -> (y fp32 [M, N], y bf16 bits)."""
    x, w = _c(x_bits, np.uint16), _c(w_hat_bits, np.uint16)
    M, K = x.shape
    N = w.shape[0]
    y32 = np.empty((M, N), dtype=np.float32)
    y16 = np.empty((M, N), dtype=np.uint16)
    lib().oracle_linear_bf16(_ptr(x), M, K, _ptr(w), N, _ptr(y32), _ptr(y16))
    return y32, y16


def moe_w4a16(x_bits, ids, wts, w13_hat, w2_hat, dumps: bool = False):
    x, ids, wts = _c(x_bits, np.uint16), _c(ids, np.int32), _c(wts, np.float32)
    w13_hat, w2_hat = _c(w13_hat, np.uint16), _c(w2_hat, np.uint16)
    M, H = x.shape
    k = ids.shape[1]
    E, I2, _ = w13_hat.shape
    I = I2 // 2
    P = M * k
    out = np.empty((M, H), dtype=np.uint16)
    d = {}
    if dumps:
        d = dict(gate_up=np.empty((P, 2 * I), np.uint16), h=np.empty((P, I), np.uint16),
                 y32=np.empty((P, H), np.float32))
    rc = lib().oracle_moe_w4a16(_ptr(x), _ptr(ids), _ptr(wts), M, H, I, E, k, _ptr(w13_hat), _ptr(w2_hat),
                                _ptr(out), _ptr(d.get("gate_up")), _ptr(d.get("h")), _ptr(d.get("y32")))
    if rc:
        raise OracleError(rc)
    return (out, d) if dumps else out


# ---------------------------------------------------------------------------- STE backward
def linear_bwd(dy_bits, x_bits, w_bits):
    """Backward of y = x . W^T on bf16 masters (straight-through past the quantizer):
    -> (dX fp32 [M, K], dX bf16 bits, dW fp32 [N, K])."""
    dy, x, w = _c(dy_bits, np.uint16), _c(x_bits, np.uint16), _c(w_bits, np.uint16)
    M, N = dy.shape
    K = x.shape[1]
    assert x.shape == (M, K) and w.shape == (N, K)
    dx32 = np.empty((M, K), dtype=np.float32)
    dx16 = np.empty((M, K), dtype=np.uint16)
    dw32 = np.empty((N, K), dtype=np.float32)
    lib().oracle_linear_bwd(_ptr(dy), _ptr(x), _ptr(w), M, N, K, _ptr(dx32), _ptr(dx16), _ptr(dw32))
    return dx32, dx16, dw32


# ---------------------------------------------------------------------------- TBPO
TBPO_DEFAULTS = dict(eps_h=4e-4, delta_l=3e-4, delta_h=7e-4, cap=2.0)   # the paper's hyper-parameter table


def tbpo(lp_cur, lp_old_learner, lp_old_sampler, offsets, adv, eps_h=4e-4, delta_l=3e-4, delta_h=7e-4, cap=2.0):
    """Sequence-level TBPO surrogate over B packed responses (offsets int64 [B+1] into the flat
    fp32 token arrays) -> dict(r, w, J float64 [B], flags int32 [B], grad fp32 [T], loss float)."""
    a, b, c = (_c(v, np.float32) for v in (lp_cur, lp_old_learner, lp_old_sampler))
    off, adv = _c(offsets, np.int64), _c(adv, np.float32)
    B = adv.shape[0]
    T = a.shape[0]
    assert off.shape == (B + 1,) and off[0] == 0 and off[-1] == T and b.shape == c.shape == (T,)
    r, w, J = (np.empty(B, dtype=np.float64) for _ in range(3))
    flags = np.empty(B, dtype=np.int32)
    grad = np.zeros(T, dtype=np.float32)
    loss = np.zeros(1, dtype=np.float64)
    lib().oracle_tbpo(_ptr(a), _ptr(b), _ptr(c), _ptr(off), _ptr(adv), B, eps_h, delta_l, delta_h, cap,
                      _ptr(r), _ptr(w), _ptr(J), _ptr(flags), _ptr(grad), _ptr(loss))
    return dict(r=r, w=w, J=J, flags=flags, grad=grad, loss=float(loss[0]))


# ---------------------------------------------------------------------------- router
def router_topk(logits, k: int):
    """fp32 logits [M, E] -> (ids int32 [M, k] in descending-logit order, ties to the lower id;
    weights fp32 [M, k] = softmax over the selected logits)."""
    l = _c(logits, np.float32)
    M, E = l.shape
    assert 1 <= k <= E
    ids = np.empty((M, k), dtype=np.int32)
    wts = np.empty((M, k), dtype=np.float32)
    lib().oracle_router_topk(_ptr(l), M, E, k, _ptr(ids), _ptr(wts))
    return ids, wts


def router(x_bits, w_router_bits, k: int):
    """Router forward: logits = x . W_r^T (bf16 operands, exact sum -> fp32), then router_topk."""
    logits, _ = linear_bf16(x_bits, w_router_bits)
    ids, wts = router_topk(logits, k)
    return logits, ids, wts


def grouped_linear_bwd(dy_bits, x_bits, w_bits, offsets):
    """linear_bwd per expert on expert-sorted rows: dy [P, N], x [P, K], w [E, N, K], offsets [E+1]
    -> (dX fp32 [P, K], dX bf16 bits, dW fp32 [E, N, K]); an expert without rows has dW = 0."""
    dy, x, w = _c(dy_bits, np.uint16), _c(x_bits, np.uint16), _c(w_bits, np.uint16)
    P, K = x.shape
    E, N, _ = w.shape
    dx32 = np.zeros((P, K), dtype=np.float32)
    dx16 = np.zeros((P, K), dtype=np.uint16)
    dw32 = np.zeros((E, N, K), dtype=np.float32)
    for e in range(E):
        a, b = int(offsets[e]), int(offsets[e + 1])
        if b > a:
            dx32[a:b], dx16[a:b], dw32[e] = linear_bwd(dy[a:b], x[a:b], w[e])
    return dx32, dx16, dw32


# ---------------------------------------------------------------------------- MoE layer backward
def swiglu_bwd(gate_up_bits, dh_bits) -> np.ndarray:
    """gate_up bf16 [P, 2I] (saved by the forward), dH bf16 [P, I] -> dGU bf16 bits [P, 2I]."""
    gu, dh = _c(gate_up_bits, np.uint16), _c(dh_bits, np.uint16)
    P, I2 = gu.shape
    out = np.empty((P, I2), dtype=np.uint16)
    lib().oracle_swiglu_bwd(_ptr(gu), _ptr(dh), P, I2 // 2, _ptr(out))
    return out


def _bf16f(bits):
    return (np.ascontiguousarray(bits, dtype=np.uint16).astype(np.uint32) << 16).view(np.float32)


def moe_bwd(x_bits, ids, wts, w13_bits, w2_bits, gate_up_bits, h_bits, dout_bits, y32=None):
    """Full-precision backward of the routed MoE FFN layer (straight-through past both quantizers) on
    the bf16 masters w13 [E, 2I, H], w2 [E, H, I] and the bf16 activations the low-bit forward saved
    in expert-sorted order (gate_up [P, 2I], h [P, I]); dout bf16 [M, H].  Steps, each rounding its
    result to bf16 where a tensor crosses an op boundary:
      dy[q]  = bf16(w_pair * dout[token])                      per sorted pair q
      dH     = bf16(dy . W2_e),     dW2_e  = dy^T h            (fp32)
      dGU    = swiglu_bwd(gate_up, dH)
      dXs    = bf16(dGU . W13_e),   dW13_e = dGU^T x_sorted    (fp32)
      dX[t]  = bf16(sum of the token's k rows of dXs in ascending expert id)
      dwts[t, j] = <dout[t], y32[q]>  (fp32; only if the forward's fp32 down output y32 [P, H], sorted, is given)
    Returns dict(dx bf16 bits [M, H], dw13, dw2 fp32, dwts or None, and the intermediates)."""
    ids, wts = _c(ids, np.int32), _c(wts, np.float32)
    M, k = ids.shape
    E = w13_bits.shape[0]
    off, srt, pos = permute(ids, E)
    tok = srt // k
    dout = _bf16f(dout_bits)
    dy = bf16_rne((wts.reshape(-1)[srt][:, None] * dout[tok]).astype(np.float32))
    x_sorted = _c(x_bits, np.uint16)[tok]
    _, dh16, dw2 = grouped_linear_bwd(dy, h_bits, w2_bits, off)
    dgu = swiglu_bwd(gate_up_bits, dh16)
    _, dxs16, dw13 = grouped_linear_bwd(dgu, x_sorted, w13_bits, off)
    by_pair = np.empty((M * k, dxs16.shape[1]), dtype=np.float32)
    by_pair[srt] = _bf16f(dxs16)
    dx = combine(by_pair, ids, np.ones_like(wts))
    dwts = None
    if y32 is not None:
        d = (dout[tok].astype(np.float64) * np.asarray(y32, dtype=np.float64)).sum(axis=1).astype(np.float32)
        dwts = np.empty(M * k, dtype=np.float32)
        dwts[srt] = d
        dwts = dwts.reshape(M, k)
    return dict(dx=dx, dw13=dw13, dw2=dw2, dwts=dwts, dy=dy, dh=dh16, dgu=dgu, dxs=dxs16, offsets=off, sorted_pair=srt)
