"""Pins for the oracle's W4A16 path (Sec. 2.2, integer quantization: W_q = clamp(round(W/s) + z,
q_min, q_max), W^ = s (W_q - z); weight-only 4-bit with bf16 activations)."""
import numpy as np
import pytest

import oracle
from paper_2604_07853_b200 import inputs


def _unpack(packed):
    lo, hi = packed & 15, packed >> 4
    return np.stack([lo, hi], axis=-1).reshape(*packed.shape[:-1], packed.shape[-1] * 2)


def _bf16_round(a):
    """fp32 -> nearest bf16 (ties to even), by integer arithmetic on the bit pattern."""
    u = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32).astype(np.uint64)
    u = (u + 0x7FFF + ((u >> 16) & 1)) & 0xFFFF0000
    return u.astype(np.uint32).view(np.float32)


def test_hand_worked_group_follows_the_paper_formula():
    """Values k/4 for k = -8..7 repeated: lo = -2, hi = 1.75, s = 3.75/15 = 0.25, z = round(2/0.25) = 8,
    W_q = W/s + 8 = 0..15 exactly and s (W_q - z) reproduces W exactly."""
    vals = (np.arange(-8, 8) / 4.0).astype(np.float32)
    w = np.tile(vals, 8)[None, :]                                  # one row, one group of 128
    p, s, z = oracle.quantize_weight_w4(inputs.f32_to_bf16_bits(w))
    assert s.shape == (1, 1) and s[0, 0] == np.float32(0.25) and z[0, 0] == 8
    q = _unpack(p)
    assert np.array_equal(q[0], np.tile(np.arange(16), 8))
    assert p[0, 0] == (0 | (1 << 4))                               # even k in the low nibble
    what = inputs.bf16_bits_to_f32(oracle.dequant_w4(p, s, z))
    assert np.array_equal(what, w)


def test_codes_scales_zeros_vs_independent_numpy():
    rng = np.random.default_rng(0)
    w = inputs.weight_bf16(rng, 3, 96, 384)
    wf = inputs.bf16_bits_to_f32(w).reshape(3, 96, 3, 128)
    p, s, z = oracle.quantize_weight_w4(w)
    lo = np.minimum(wf.min(axis=3), 0).astype(np.float32)
    hi = np.maximum(wf.max(axis=3), 0).astype(np.float32)
    s_ref = (np.maximum(hi - lo, np.float32(2.0 ** -40)) / np.float32(15)).astype(np.float32)
    s_ref = _bf16_round(s_ref)                                     # the scale is stored as bf16
    z_ref = np.clip(np.rint((-lo / s_ref).astype(np.float32)), 0, 15)
    assert np.array_equal(s, s_ref) and np.array_equal(z, z_ref.astype(np.uint8))
    q_ref = np.clip(np.rint((wf / s_ref[..., None]).astype(np.float32)) + z_ref[..., None], 0, 15)
    q = _unpack(p).reshape(3, 96, 3, 128)
    assert np.array_equal(q, q_ref.astype(np.uint8))
    assert q.min() >= 0 and q.max() <= 15
    # every group uses the full range: its min maps to 0 or its max to 15 (usually both)
    assert ((q.min(axis=3) == 0) | (q.max(axis=3) == 15)).all()


def test_round_trip_bound_and_exact_zero():
    rng = np.random.default_rng(1)
    w = inputs.weight_bf16(rng, 64, 512)
    w[:, ::7] = 0                                                  # exact zeros
    w[5, :128] = 0                                                 # an all-zero group
    p, s, z = oracle.quantize_weight_w4(w)
    wf = inputs.bf16_bits_to_f32(w).astype(np.float64)
    what = inputs.bf16_bits_to_f32(oracle.dequant_w4(p, s, z)).astype(np.float64)
    se = np.repeat(s, 128, axis=1).astype(np.float64)
    q = _unpack(p).astype(np.int64)
    inner = (q > 0) & (q < 15)                                     # codes that were not clamped
    # half a step from rounding, plus the bf16 rounding of the dequantized value
    bound = 0.5 * se * (1 + 1e-5) + np.abs(what) * 2.0 ** -8
    assert (np.abs(wf - what)[inner] <= bound[inner]).all()
    # clamped codes: the rounded zero point and the bf16-rounded scale add at most one more step
    assert (np.abs(wf - what) <= bound + se * (0.5 + 16 * 2.0 ** -8)).all()
    assert (what[wf == 0] == 0).all()                              # zero is representable (code z)
    assert np.array_equal(s, _bf16_round(s))                       # scales are bf16 values
    assert np.isfinite(s).all() and s[5, 0] == _bf16_round(np.float32(2.0 ** -40) / np.float32(15))


def test_dequant_is_bf16_of_one_fp32_product():
    rng = np.random.default_rng(2)
    p = rng.integers(0, 256, size=(16, 64), dtype=np.uint8)
    s = rng.uniform(1e-3, 1e-1, size=(16, 1)).astype(np.float32)
    z = rng.integers(0, 16, size=(16, 1), dtype=np.uint8)
    q = _unpack(p).astype(np.int32)
    ref = inputs.f32_to_bf16_bits((s * (q - z.astype(np.int32)).astype(np.float32)).astype(np.float32))
    assert np.array_equal(oracle.dequant_w4(p, s, z), ref)


def test_linear_bf16_vs_float64_and_exact_case():
    rng = np.random.default_rng(3)
    x = inputs.act_bf16(rng, 9, 256)
    w = inputs.weight_bf16(rng, 40, 256)
    y32, y16 = oracle.linear_bf16(x, w)
    ref = inputs.bf16_bits_to_f32(x).astype(np.float64) @ inputs.bf16_bits_to_f32(w).astype(np.float64).T
    assert np.array_equal(y32, ref.astype(np.float32))             # exact sum, one rounding
    assert np.array_equal(y16, inputs.f32_to_bf16_bits(y32))
    xi = inputs.f32_to_bf16_bits(rng.integers(-8, 9, size=(4, 128)).astype(np.float32))
    wi = inputs.f32_to_bf16_bits(rng.integers(-8, 9, size=(6, 128)).astype(np.float32))
    yi, _ = oracle.linear_bf16(xi, wi)
    assert np.array_equal(yi, (inputs.bf16_bits_to_f32(xi) @ inputs.bf16_bits_to_f32(wi).T))


def test_moe_w4a16_composition_and_closeness_to_unquantized():
    c = inputs.moe_case(5, 12, h=256, i=128, e=4, k=2)
    w13h = oracle.dequant_w4(*oracle.quantize_weight_w4(c.w13))
    w2h = oracle.dequant_w4(*oracle.quantize_weight_w4(c.w2))
    out, d = oracle.moe_w4a16(c.x, c.ids, c.weights, w13h, w2h, dumps=True)
    assert np.array_equal(d["h"], oracle.swiglu(d["gate_up"]))
    assert np.array_equal(out, oracle.combine(d["y32"], c.ids, c.weights))
    for p in range(0, c.M * c.k, 5):
        t, e = p // c.k, c.ids.reshape(-1)[p]
        _, gu = oracle.linear_bf16(c.x[t:t + 1], w13h[e])
        assert np.array_equal(gu[0], d["gate_up"][p])
        y32, _ = oracle.linear_bf16(d["h"][p:p + 1], w2h[e])
        assert np.array_equal(y32[0], d["y32"][p])
    xf = inputs.bf16_bits_to_f32(c.x).astype(np.float64)
    w13 = inputs.bf16_bits_to_f32(c.w13).astype(np.float64)
    w2 = inputs.bf16_bits_to_f32(c.w2).astype(np.float64)
    ref = np.zeros((c.M, c.H))
    for t in range(c.M):
        for j in range(c.k):
            e = c.ids[t, j]
            gu = w13[e] @ xf[t]
            g, u = gu[:c.I], gu[c.I:]
            ref[t] += c.weights[t, j] * (w2[e] @ (g / (1 + np.exp(-g)) * u))
    got = inputs.bf16_bits_to_f32(out).astype(np.float64)
    rel = np.linalg.norm(got - ref) / np.linalg.norm(ref)
    assert 0.01 < rel < 0.25           # 4-bit weights: visible but bounded quantization noise


def test_w4_shape_error():
    with pytest.raises(oracle.OracleError):
        oracle.quantize_weight_w4(np.zeros((4, 100), np.uint16))
