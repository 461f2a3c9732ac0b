"""Pins for the oracle's block-scaled linear (Sec. 2.2: Y ~= (s_x s_w)(X_q W_q), applied per
128-wide K-block with higher-precision accumulation)."""
import ml_dtypes
import numpy as np
import torch

import oracle
from paper_2604_07853_b200 import inputs

F8 = ml_dtypes.float8_e4m3fn
DEC = np.arange(256, dtype=np.uint8).view(F8).astype(np.float64)


def _blockwise_f64(xc, xs, wc, ws):
    """Independent restatement in float64 with library decode: sum_kb s_x s_w (x_q . w_q)."""
    M, K = xc.shape
    N = wc.shape[0]
    kb = K // 128
    xd = DEC[xc].reshape(M, kb, 128)
    wd = DEC[wc].reshape(N, kb, 128)
    p = np.einsum("mbk,nbk->mnb", xd, wd)                       # exact in float64
    sc = xs.astype(np.float64)[:, None, :] * np.repeat(ws.astype(np.float64), 128, axis=0)[None]
    return (p * sc).sum(axis=2), np.abs(p * sc).sum(axis=2)


def test_exact_special_case_equals_fp64_unquantized_product():
    """Inputs built so that quantization is lossless and every partial sum is an integer
    below 2^24: the oracle must equal the float64 product of the ORIGINAL tensors exactly."""
    rng = np.random.default_rng(0)
    M, N, K = 24, 256, 384
    kb = K // 128
    ax = rng.integers(-6, 7, size=(M, kb))            # per-group exponents of x
    aw = rng.integers(-6, 7, size=(N // 128, kb))     # per-block exponents of w
    x = rng.integers(-8, 9, size=(M, K)).astype(np.float64)
    w = rng.integers(-8, 9, size=(N, K)).astype(np.float64)
    for m in range(M):
        for b in range(kb):
            x[m, b * 128 + rng.integers(128)] = 448.0 * rng.choice([-1, 1])
    for bn in range(N // 128):
        for b in range(kb):
            w[bn * 128 + rng.integers(128), b * 128 + rng.integers(128)] = 448.0 * rng.choice([-1, 1])
    x *= 2.0 ** np.repeat(ax, 128, axis=1)
    w *= 2.0 ** np.repeat(np.repeat(aw, 128, axis=0), 128, axis=1)
    xb, wb = inputs.f32_to_bf16_bits(x), inputs.f32_to_bf16_bits(w)
    assert np.array_equal(inputs.bf16_bits_to_f32(xb).astype(np.float64), x)   # bf16-exact inputs
    assert np.array_equal(inputs.bf16_bits_to_f32(wb).astype(np.float64), w)
    wc, ws = oracle.quantize_weight(wb)
    xc, xs = oracle.quantize_act(xb)
    assert np.array_equal(xs, (2.0 ** ax).astype(np.float32))
    assert np.array_equal(ws, (2.0 ** aw).astype(np.float32))
    assert np.array_equal(DEC[xc] * np.repeat(xs, 128, axis=1), x)             # lossless
    y32, y16 = oracle.linear(xb, wc, ws)
    ref = x @ w.T
    # block sums are integers < 2^24 times a power of two, but the kb-chain may round once
    # the magnitudes of different blocks differ; restrict the bit-exact claim to rows and
    # columns whose blocks share one exponent, and bound the rest by fp32 rounding
    same = (ax.max(axis=1) == ax.min(axis=1))[:, None] & \
           np.repeat(aw.max(axis=1) == aw.min(axis=1), 128)[None, :]
    assert np.array_equal(y32[same].astype(np.float64), ref[same])
    assert np.allclose(y32, ref, rtol=2.0 ** -21, atol=0)
    t16 = torch.from_numpy(y32).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(y16, t16)


def test_exact_case_single_exponent_everywhere_bitwise():
    rng = np.random.default_rng(1)
    M, N, K = 16, 128, 512
    x = rng.integers(-8, 9, size=(M, K)).astype(np.float64)
    w = rng.integers(-8, 9, size=(N, K)).astype(np.float64)
    x[:, ::128] = 448.0
    w[3, ::128] = -448.0
    x *= 2.0 ** -3
    w *= 2.0 ** 2
    xb, wb = inputs.f32_to_bf16_bits(x), inputs.f32_to_bf16_bits(w)
    wc, ws = oracle.quantize_weight(wb)
    y32, _ = oracle.linear(xb, wc, ws)
    assert np.array_equal(y32.astype(np.float64), x @ w.T)


def test_single_block_reduces_to_paper_per_tensor_formula():
    """K = 128, N = 128: one scale per operand row / matrix, so the result is exactly
    (s_x s_w) (X_q W_q) rounded to fp32 (the paper's low-bit GEMM equation)."""
    c = inputs.linear_case(11, 8, 128, 128)
    wc, ws = oracle.quantize_weight(c.w)
    xc, xs = oracle.quantize_act(c.x)
    y32, _ = oracle.linear_q(xc, xs, wc, ws)
    p = (DEC[xc] @ DEC[wc].T).astype(np.float32)                  # exact dot, one rounding
    sc = (xs * ws[0, 0]).astype(np.float32)                        # [M,1]
    ref = (sc.astype(np.float64) * p.astype(np.float64)).astype(np.float32)
    assert np.array_equal(y32, ref)


def test_general_vs_float64_blockwise_restatement():
    c = inputs.linear_case(12, 40, 384, 640)                       # M, N, K all different
    wc, ws = oracle.quantize_weight(c.w)
    xc, xs = oracle.quantize_act(c.x)
    y32, y16 = oracle.linear_q(xc, xs, wc, ws)
    ref, mag = _blockwise_f64(xc, xs, wc, ws)
    assert (np.abs(y32 - ref) <= mag * 2.0 ** -21 + 1e-30).all()
    # and linear() == quantize_act + linear_q
    y32b, y16b = oracle.linear(c.x, wc, ws)
    assert np.array_equal(y32, y32b) and np.array_equal(y16, y16b)


def test_config1_vs_fp64_unquantized_within_propagated_bound():
    c = inputs.config1()
    xf = inputs.bf16_bits_to_f32(c.x).astype(np.float64)
    wf = inputs.bf16_bits_to_f32(c.w).astype(np.float64)
    wc, ws = oracle.quantize_weight(c.w)
    xc, xs = oracle.quantize_act(c.x)
    y32, _ = oracle.linear_q(xc, xs, wc, ws)
    sx = np.repeat(xs, 128, axis=1).astype(np.float64)
    sw = np.repeat(np.repeat(ws, 128, axis=0), 128, axis=1).astype(np.float64)
    dx = np.maximum(np.abs(xf) * 2.0 ** -4, sx * 2.0 ** -10)
    dw = np.maximum(np.abs(wf) * 2.0 ** -4, sw * 2.0 ** -10)
    bound = np.abs(xf) @ dw.T + dx @ np.abs(wf).T + dx @ dw.T
    ref = xf @ wf.T
    slack = (np.abs(xf) @ np.abs(wf).T) * 2.0 ** -20
    assert (np.abs(y32 - ref) <= bound + slack).all()
    rel = np.linalg.norm(y32 - ref) / np.linalg.norm(ref)
    assert 0.005 < rel < 0.06          # quantization noise is present and of the expected size


def test_scale_indexing_is_not_symmetric():
    """A wrong scale index (n vs n/128, kb swapped) must change the result: use scales that
    differ strongly across blocks and compare with the float64 restatement."""
    rng = np.random.default_rng(13)
    M, N, K = 5, 256, 256
    xc = rng.integers(0, 0x7F, size=(M, K)).astype(np.uint8)
    wc = rng.integers(0, 0x7F, size=(N, K)).astype(np.uint8)
    xs = (2.0 ** rng.integers(-8, 8, size=(M, 2))).astype(np.float32)
    ws = (2.0 ** rng.integers(-8, 8, size=(2, 2))).astype(np.float32)
    y32, _ = oracle.linear_q(xc, xs, wc, ws)
    ref, mag = _blockwise_f64(xc, xs, wc, ws)
    assert (np.abs(y32 - ref) <= mag * 2.0 ** -22).all()
