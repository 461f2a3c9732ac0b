"""Pins for the oracle's casts: e4m3 decode / encode and bf16 rounding.

None of these re-type the oracle's formula: they compare against independent library casts
(ml_dtypes, torch), the format's closed-form facts, the constant the paper prints, and a
brute-force nearest-value search."""
import os

import ml_dtypes
import numpy as np
import torch

import oracle

F8 = ml_dtypes.float8_e4m3fn
GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "paper_constants.txt")


def _golden():
    out = {}
    for line in open(GOLDEN):
        if line.strip() and not line.startswith("#"):
            k, v = line.split()
            out[k] = float(v)
    return out


def test_decode_table_matches_library_and_paper_alpha():
    tab = oracle.e4m3_decode_table()
    ref = np.arange(256, dtype=np.uint8).view(F8).astype(np.float64)
    assert np.array_equal(np.isnan(tab), np.isnan(ref))
    fin = ~np.isnan(tab)
    assert np.array_equal(tab[fin], ref[fin])
    assert np.array_equal(np.signbit(tab[fin]), np.signbit(ref[fin]))
    # format facts: 254 finite codes, NaN only at 0x7F / 0xFF, max = alpha (paper, Sec. 2.2)
    assert fin.sum() == 254 and list(np.where(~fin)[0]) == [0x7F, 0xFF]
    assert tab[fin].max() == _golden()["alpha_e4m3"] == tab[0x7E]
    assert tab[0x01] == 2.0 ** -9 and tab[0x08] == 2.0 ** -6
    # monotone in the code for each sign
    assert np.all(np.diff(tab[0:0x7F]) > 0)
    assert np.all(np.diff(tab[0x80:0xFF]) < 0)


def _lib_cast(v: np.ndarray) -> np.ndarray:
    """Independent cast: clamp to +-448 (saturation), then ml_dtypes RNE cast."""
    return np.clip(v, -448.0, 448.0).astype(F8).view(np.uint8)


def test_encode_structured_patterns_vs_ml_dtypes():
    # every fp32 exponent/upper-mantissa pattern with low mantissa bytes that sit on, just
    # below and just above every rounding boundary
    hi = np.arange(0, 1 << 16, dtype=np.uint32) << 16          # sign, exponent, 7 mantissa bits
    lows = np.array([0x0000, 0x0001, 0x7FFF, 0x8000, 0x8001, 0xFFFF, 0x4000, 0xC000,
                     0x0FFF, 0x1000, 0x1001, 0xEFFF, 0xF000, 0xF001], dtype=np.uint32)
    bits = (hi[:, None] | lows[None, :]).reshape(-1)
    v = bits.view(np.float32)
    ok = np.isfinite(v)
    v = v[ok]
    assert np.array_equal(oracle.e4m3_encode(v), _lib_cast(v))


def test_encode_random_bit_patterns_vs_torch_and_ml_dtypes():
    rng = np.random.default_rng(1)
    bits = rng.integers(0, 1 << 32, size=8_000_000, dtype=np.uint64).astype(np.uint32)
    v = bits.view(np.float32)
    v = v[np.isfinite(v)]
    got = oracle.e4m3_encode(v)
    assert np.array_equal(got, _lib_cast(v))
    t = torch.from_numpy(v).clamp(-448.0, 448.0).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    assert np.array_equal(got, t)


def test_encode_dense_sweep_near_grid():
    # values within the e4m3 range, dense around every grid point and midpoint
    tab = oracle.e4m3_decode_table()[:0x7F]
    mids = (tab[:-1] + tab[1:]) / 2
    pts = np.concatenate([tab, mids]).astype(np.float32)
    eps = np.array([-3, -2, -1, 0, 1, 2, 3])
    bits = (pts.view(np.uint32).astype(np.int64)[:, None] + eps[None, :]).clip(0).astype(np.uint32)
    v = bits.reshape(-1).view(np.float32)
    v = np.concatenate([v, -v])
    assert np.array_equal(oracle.e4m3_encode(v), _lib_cast(v))


def test_encode_is_nearest_value_ties_to_even_code_brute_force():
    rng = np.random.default_rng(2)
    tab = oracle.e4m3_decode_table()
    pos = tab[:0x7F]                       # 127 non-negative finite values, ascending
    v = np.concatenate([rng.uniform(-500, 500, 50_000), rng.standard_normal(50_000) * 0.01,
                        rng.standard_normal(50_000) * 4.0, (pos[:-1] + pos[1:]) / 2,
                        -(pos[:-1] + pos[1:]) / 2]).astype(np.float32)
    a = np.abs(v.astype(np.float64))
    d = np.abs(a[:, None] - pos[None, :])
    best = d.min(axis=1)
    cand = d == best[:, None]              # one or two nearest codes
    idx = np.arange(127)[None, :]
    even = (idx % 2 == 0)
    pick_even = np.where(cand & even, idx, -1).max(axis=1)
    pick_any = np.where(cand, idx, -1).max(axis=1)
    ties = cand.sum(axis=1) == 2
    code = np.where(ties, pick_even, pick_any)
    code = np.where(a > 448, 0x7E, code).astype(np.uint8)
    code |= (np.signbit(v).astype(np.uint8) << 7)
    assert np.array_equal(oracle.e4m3_encode(v), code)


def test_encode_special_cases():
    enc = oracle.e4m3_encode
    assert list(enc([0.0, -0.0])) == [0x00, 0x80]
    assert list(enc([448.0, 464.0, 479.9, 480.0, 1e30, -1e30])) == [0x7E] * 5 + [0xFE]
    assert list(enc([2.0 ** -10, 3 * 2.0 ** -10, -1e-9])) == [0x00, 0x02, 0x80]  # ties, underflow
    assert list(enc([2.0 ** -10 * 1.0001])) == [0x01]


def test_bf16_rne_vs_torch():
    rng = np.random.default_rng(3)
    bits = rng.integers(0, 1 << 32, size=4_000_000, dtype=np.uint64).astype(np.uint32)
    hi = np.arange(0, 1 << 16, dtype=np.uint32) << 16
    lows = np.array([0, 1, 0x7FFF, 0x8000, 0x8001, 0xFFFF], dtype=np.uint32)
    bits = np.concatenate([bits, (hi[:, None] | lows[None, :]).reshape(-1)])
    v = bits.view(np.float32)
    v = v[np.isfinite(v)]
    ref = torch.from_numpy(v).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(oracle.bf16_rne(v), ref)


def test_encode_every_fp32_bit_pattern_vs_torch_cast():
    """All 2^32 fp32 bit patterns (the finite ones: NaN and infinity are outside the contract) through
    the oracle's encoder and through torch's float8_e4m3fn cast after an explicit clamp to +-448
    (the cast rounds to nearest even; the clamp is the saturation the reading adds)."""
    n = 1 << 26
    checked = 0
    for base in range(0, 1 << 32, n):
        v = np.arange(base, base + n, dtype=np.uint64).astype(np.uint32).view(np.float32)
        fin = np.isfinite(v)
        if not fin.all():
            v = v[fin]
        got = oracle.e4m3_encode(v)
        ref = torch.from_numpy(v).clamp(-448.0, 448.0).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
        assert np.array_equal(got, ref), hex(base)
        checked += v.size
    assert checked == (1 << 32) - (1 << 24)              # everything but the two exponent-255 ranges (2 x 2^23)
