"""Pins for the oracle's FP4 (e2m1) weight-only path (Sec. 2.2, floating-point quantization:
s = max|W| / alpha, W_q = [W / s]_FP4, W^ = s W_q, alpha = 6 for e2m1)."""
import numpy as np
import pytest

import oracle
from paper_2604_07853_b200 import inputs

MAGNITUDES = [0.0, 0.5, 1.0, 1.5, 2.0, 3.0, 4.0, 6.0]   # sign, 2 exponent bits (bias 1), 1 mantissa bit


def _unpack(packed):
    lo, hi = packed & 15, packed >> 4
    return np.stack([lo, hi], axis=-1).reshape(*packed.shape[:-1], packed.shape[-1] * 2)


def _bf16_round(a):
    """fp32 -> nearest bf16 (ties to even), by integer arithmetic on the bit pattern."""
    u = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32).astype(np.uint64)
    u = (u + 0x7FFF + ((u >> 16) & 1)) & 0xFFFF0000
    return u.astype(np.uint32).view(np.float32)


def test_code_table_and_alpha():
    """Sec. 2.2: alpha is the largest finite value of the format, 6 for e2m1."""
    t = oracle.e2m1_table()
    assert t[:8].tolist() == MAGNITUDES
    assert t[8:].tolist() == [-m for m in MAGNITUDES] and np.signbit(t[8])
    assert np.abs(t).max() == 6.0
    # the bit fields: subnormal step 0.5, then 2^(ee-1) (1 + m/2)
    for c in range(8):
        ee, m = c >> 1, c & 1
        assert t[c] == (0.5 * m if ee == 0 else 2.0 ** (ee - 1) * (1 + 0.5 * m))


def test_encode_hand_values_and_ties_to_even():
    """Midpoints go to the neighbour whose mantissa bit is 0: 0.25->0, 0.75->1, 1.25->1, 1.75->2,
    2.5->2, 3.5->4, 5->4; beyond 6 saturates; the sign is kept, also on zero."""
    v = [0.25, 0.75, 1.25, 1.75, 2.5, 3.5, 5.0, 6.0, 7.0, 1e30, 0.0, 0.2500001, 0.7499999, 5.0000005]
    want = [0, 2, 2, 4, 4, 6, 6, 7, 7, 7, 0, 1, 1, 7]
    assert oracle.e2m1_encode(v).tolist() == want
    assert oracle.e2m1_encode([-x for x in v]).tolist() == [8 | c for c in want]


def test_encode_matches_a_library_cast():
    """An independent implementation of the same rounding: ml_dtypes' float4_e2m1fn cast
    (round to nearest even, saturating-finite format)."""
    ml_dtypes = pytest.importorskip("ml_dtypes")
    rng = np.random.default_rng(0)
    v = np.concatenate([rng.uniform(-6, 6, 20000), rng.normal(0, 1, 20000),
                        np.arange(-24, 25) / 4.0, np.arange(-48, 49) / 8.0]).astype(np.float32)
    got = oracle.e2m1_table()[oracle.e2m1_encode(v)]
    lib = v.astype(ml_dtypes.float4_e2m1fn).astype(np.float64)
    assert np.array_equal(got, lib)
    assert np.array_equal(np.signbit(got), np.signbit(lib))


def test_encode_is_nearest_monotone_and_idempotent():
    rng = np.random.default_rng(1)
    v = np.sort(rng.uniform(0, 8, 5000)).astype(np.float32)
    c = oracle.e2m1_encode(v)
    assert (np.diff(c.astype(int)) >= 0).all()
    got = oracle.e2m1_table()[c]
    table = np.array(MAGNITUDES)
    brute = np.abs(v.astype(np.float64)[:, None] - table[None, :]).min(axis=1)   # distance to the nearest value
    assert np.array_equal(np.abs(got - v.astype(np.float64)), brute)
    assert oracle.e2m1_encode(np.array(MAGNITUDES, np.float32)).tolist() == list(range(8))


def test_hand_worked_group():
    """amax = 6 gives s = 1 exactly, so the codes are the e2m1 roundings of the values themselves."""
    vals = np.array([6.0, -3.0, 2.5, 0.75, 0.25, 1.25, -1.75, 5.0, -6.0, 0.5, -0.25, 4.5, 1.0, -1.5, 3.25, 0.0],
                    dtype=np.float32)
    want = [7, 13, 4, 2, 0, 2, 12, 6, 15, 1, 8, 6, 2, 11, 5, 0]
    w = np.tile(vals, 8)[None, :]
    p, s = oracle.quantize_weight_fp4(inputs.f32_to_bf16_bits(w))
    assert s.shape == (1, 1) and s[0, 0] == np.float32(1.0)
    assert _unpack(p)[0].tolist() == want * 8
    assert p[0, 0] == (7 | (13 << 4))                              # even k in the low nibble
    what = inputs.bf16_bits_to_f32(oracle.dequant_fp4(p, s))
    assert np.array_equal(what[0, :16], oracle.e2m1_table()[want].astype(np.float32))


def test_scales_and_codes_vs_independent_numpy():
    ml_dtypes = pytest.importorskip("ml_dtypes")
    rng = np.random.default_rng(2)
    w = inputs.weight_bf16(rng, 3, 96, 384)
    wf = inputs.bf16_bits_to_f32(w).reshape(3, 96, 3, 128)
    p, s = oracle.quantize_weight_fp4(w)
    amax = np.maximum(np.abs(wf).max(axis=3), np.float32(2.0 ** -40))
    s_ref = _bf16_round((amax / np.float32(6)).astype(np.float32))
    assert np.array_equal(s, s_ref)
    t = (wf / s_ref[..., None]).astype(np.float32)
    q_val = t.astype(ml_dtypes.float4_e2m1fn).astype(np.float64)
    q = _unpack(p).reshape(3, 96, 3, 128)
    assert np.array_equal(oracle.e2m1_table()[q], q_val)
    # the group maximum always lands on +-6: s differs from amax/6 by at most 2^-9 relative
    assert (np.abs(oracle.e2m1_table()[q]).max(axis=3) == 6.0).all()
    # dequantized weight = bf16(s * value), the product formed exactly
    what = inputs.bf16_bits_to_f32(oracle.dequant_fp4(p, s)).reshape(3, 96, 3, 128)
    exact = s_ref[..., None].astype(np.float64) * q_val
    assert np.array_equal(what, _bf16_round(exact.astype(np.float32)))   # exact fits fp32: 8 + 2 bits


def test_round_trip_bound_zero_group_and_symmetries():
    rng = np.random.default_rng(3)
    w = inputs.weight_bf16(rng, 64, 512)
    w[:, ::7] = 0
    w[5, :128] = 0                                                 # an all-zero group
    wf = inputs.bf16_bits_to_f32(w)
    p, s = oracle.quantize_weight_fp4(w)
    what = inputs.bf16_bits_to_f32(oracle.dequant_fp4(p, s))
    # the widest gap between neighbours is 2 (4 -> 6): |W/s - value| <= 1, plus the bf16 rounding of w^
    sg = np.repeat(s, 128, axis=1)
    assert (np.abs(wf - what) <= sg * (1.0 + 2.0 ** -7) + 1e-30).all()
    assert (what[wf == 0] == 0).all()
    assert s[5, 0] == _bf16_round(np.float32(2.0 ** -40) / np.float32(6)) and (_unpack(p)[5, :128] == 0).all()
    # sign symmetry: -W flips bit 3 of every code and leaves the scales alone
    p2, s2 = oracle.quantize_weight_fp4(w ^ np.uint16(0x8000))
    assert np.array_equal(s2, s) and np.array_equal(_unpack(p2), _unpack(p) ^ 8)
    # power-of-two covariance: 4 W has the same codes and 4 s
    w4 = inputs.f32_to_bf16_bits(wf * 4)
    p4, s4 = oracle.quantize_weight_fp4(w4)
    keep = s > 2.0 ** -30                                          # groups above the amax floor
    assert np.array_equal(s4[keep], 4 * s[keep])
    assert np.array_equal(_unpack(p4).reshape(64, 4, 128)[keep], _unpack(p).reshape(64, 4, 128)[keep])
    # groups are independent: changing one leaves the others' codes and scales alone
    w_mod = w.copy()
    w_mod[:, 128:256] = inputs.weight_bf16(rng, 64, 128)
    p3, s3 = oracle.quantize_weight_fp4(w_mod)
    other = np.r_[0:128, 256:512]
    assert np.array_equal(_unpack(p3)[:, other], _unpack(p)[:, other]) and np.array_equal(s3[:, [0, 2, 3]], s[:, [0, 2, 3]])


def test_linear_with_fp4_weights_is_the_plain_matmul_of_dequantized_weights():
    rng = np.random.default_rng(4)
    x = inputs.act_bf16(rng, 9, 256)
    w = inputs.weight_bf16(rng, 24, 256)
    p, s = oracle.quantize_weight_fp4(w)
    w_hat = oracle.dequant_fp4(p, s)
    y32, y16 = oracle.linear_bf16(x, w_hat)
    ref = inputs.bf16_bits_to_f32(x).astype(np.float64) @ inputs.bf16_bits_to_f32(w_hat).astype(np.float64).T
    assert np.array_equal(y32, ref.astype(np.float32))
    assert np.array_equal(y16, inputs.f32_to_bf16_bits(y32))
