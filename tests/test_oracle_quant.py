"""Pins for the oracle's block quantizers (Sec. 2.2: s = max|W| / alpha, W_q = [W / s]_FP8,
W^ = s * W_q with alpha = 448)."""
import ml_dtypes
import numpy as np
import pytest

import oracle
from paper_2604_07853_b200 import inputs

F8 = ml_dtypes.float8_e4m3fn
DEC = np.arange(256, dtype=np.uint8).view(F8).astype(np.float64)   # library decode table


def _roundtrip_checks(x_f32, codes, scale_per_elem):
    deq = DEC[codes] * scale_per_elem.astype(np.float64)
    err = np.abs(deq - x_f32.astype(np.float64))
    # e4m3 has 3 mantissa bits: relative error <= 2^-4 in the normal range, absolute error
    # <= half a subnormal step (s * 2^-10) below it
    bound = np.maximum(np.abs(x_f32) * 2.0 ** -4, scale_per_elem * 2.0 ** -10) * (1 + 2.0 ** -20)
    assert (err <= bound).all()
    assert not np.isnan(deq).any()
    # sign preserved wherever the code is non-zero
    nz = (codes & 0x7F) != 0
    assert np.array_equal(np.signbit(x_f32)[nz], (codes[nz] >> 7).astype(bool))


def test_act_scale_is_amax_over_alpha_and_block_hits_448():
    x = inputs.act_bf16(np.random.default_rng(0), 64, 512)
    xf = inputs.bf16_bits_to_f32(x)
    codes, scales = oracle.quantize_act(x)
    amax = np.abs(xf).reshape(64, 4, 128).max(axis=2)
    assert np.array_equal(scales, (amax / np.float32(448.0)).astype(np.float32))
    # the amax element of every group maps to +-448 (code 0x7E / 0xFE)
    g = codes.reshape(64, 4, 128) & 0x7F
    assert (g.max(axis=2) == 0x7E).all()
    where = np.abs(xf).reshape(64, 4, 128).argmax(axis=2)
    assert (np.take_along_axis(g, where[..., None], axis=2) == 0x7E).all()
    _roundtrip_checks(xf, codes, np.repeat(scales, 128, axis=1))


def test_act_codes_vs_independent_library_cast():
    x = inputs.act_bf16(np.random.default_rng(5), 32, 256)
    xf = inputs.bf16_bits_to_f32(x)
    codes, _ = oracle.quantize_act(x)
    amax = np.abs(xf).reshape(32, 2, 128).max(axis=2, keepdims=True)
    inv = np.float32(448.0) / amax
    v = (xf.reshape(32, 2, 128) * inv).astype(np.float32)
    ref = np.clip(v, -448, 448).astype(F8).view(np.uint8).reshape(32, 256)
    assert np.array_equal(codes, ref)


def test_weight_blocks_are_128x128_not_transposed():
    rng = np.random.default_rng(1)
    w = inputs.weight_bf16(rng, 2, 256, 384)           # E=2, N=256, K=384: non-square
    wf = inputs.bf16_bits_to_f32(w)
    # plant a distinct large value in each block so any block mix-up changes the scales
    for e in range(2):
        for bn in range(2):
            for bk in range(3):
                wf[e, bn * 128 + 5 + bk, bk * 128 + 7 + bn] = 1.0 + e + 2 * bn + 4 * bk
    w = inputs.f32_to_bf16_bits(wf)
    wf = inputs.bf16_bits_to_f32(w)
    codes, scales = oracle.quantize_weight(w)
    assert codes.shape == (2, 256, 384) and scales.shape == (2, 2, 3)
    amax = np.abs(wf).reshape(2, 2, 128, 3, 128).max(axis=(2, 4))
    assert np.array_equal(scales, (amax / np.float32(448.0)).astype(np.float32))
    s_elem = np.repeat(np.repeat(scales, 128, axis=1), 128, axis=2)
    _roundtrip_checks(wf, codes, s_elem)
    blk = (codes & 0x7F).reshape(2, 2, 128, 3, 128).max(axis=(2, 4))
    assert (blk == 0x7E).all()
    # 2-D convenience form equals expert 0 of the batched form
    c0, s0 = oracle.quantize_weight(w[0])
    assert np.array_equal(c0, codes[0]) and np.array_equal(s0, scales[0])


def test_zero_and_tiny_blocks():
    x = np.zeros((2, 256), dtype=np.uint16)
    x[0, 3] = 0x8000                                    # -0.0
    x[1, 130] = inputs.f32_to_bf16_bits(np.array([1e-30], np.float32))[0]   # below the floor
    codes, scales = oracle.quantize_act(x)
    floor = np.float32(2.0 ** -40) / np.float32(448.0)
    assert (scales == floor).all()
    assert codes[0, 3] == 0x80 and (np.delete(codes[0], 3) == 0).all()
    assert (codes[1] == 0).all()                        # 1e-30 * 448 * 2^40 underflows e4m3
    assert np.isfinite(scales).all()


def test_amax_maps_to_448_for_every_bf16_magnitude():
    # every positive finite bf16 in [2^-40, 2^40] as the lone non-zero of a group
    bits = np.arange(0x0080, 0x7F80, dtype=np.uint16)
    f = inputs.bf16_bits_to_f32(bits)
    bits = bits[(f >= 2.0 ** -40) & (f <= 2.0 ** 40)]
    x = np.zeros((bits.size, 128), dtype=np.uint16)
    x[:, 17] = bits
    x[::2, 17] |= 0x8000
    codes, scales = oracle.quantize_act(x)
    assert (codes[1::2, 17] == 0x7E).all() and (codes[::2, 17] == 0xFE).all()
    assert np.array_equal(scales[:, 0], inputs.bf16_bits_to_f32(bits) / np.float32(448.0))


def test_row_stride_and_shape_errors():
    x = inputs.act_bf16(np.random.default_rng(7), 4, 128)
    with pytest.raises(oracle.OracleError):
        oracle.quantize_act(x[:, :100])
    with pytest.raises(oracle.OracleError):
        oracle.quantize_weight(np.zeros((100, 128), np.uint16))
