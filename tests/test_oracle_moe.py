"""Pins for the oracle's MoE pieces: expert permutation, SwiGLU, top-k combine and the
composed layer."""
import ml_dtypes
import numpy as np
import pytest
import torch

import oracle
from paper_2604_07853_b200 import inputs

F8 = ml_dtypes.float8_e4m3fn
DEC = np.arange(256, dtype=np.uint8).view(F8).astype(np.float64)


def _ulp_dist(a_bits, b_bits):
    """Distance between bf16 values counted in representable steps."""
    def key(b):
        b = b.astype(np.int32)
        return np.where(b & 0x8000, -(b & 0x7FFF), b & 0x7FFF)
    return np.abs(key(a_bits) - key(b_bits))


def test_permute_vs_brute_force_stable_sort():
    rng = np.random.default_rng(0)
    for (m, e, k) in [(1, 4, 2), (37, 16, 4), (300, 128, 8), (64, 8, 8)]:
        ids, _ = inputs.routing(rng, m, e, k)
        off, srt, pos = oracle.permute(ids, e)
        flat = ids.reshape(-1)
        ref = np.argsort(flat, kind="stable").astype(np.int32)
        assert np.array_equal(srt, ref)
        cnt = np.bincount(flat, minlength=e)
        assert np.array_equal(off, np.concatenate([[0], np.cumsum(cnt)]).astype(np.int32))
        assert np.array_equal(pos[srt], np.arange(m * k, dtype=np.int32))
        assert off[-1] == m * k and (np.diff(off) >= 0).all()


def test_permute_rejects_bad_ids():
    ids = np.array([[0, 1], [2, 2]], dtype=np.int32)          # duplicate expert in a token
    with pytest.raises(oracle.OracleError) as ei:
        oracle.permute(ids, 4)
    assert ei.value.code == -8
    for bad in (-1, 4):
        ids = np.array([[0, bad]], dtype=np.int32)
        with pytest.raises(oracle.OracleError):
            oracle.permute(ids, 4)


def test_routing_weights_sum_to_one():
    ids, w = inputs.routing(np.random.default_rng(1), 512, 128, 8)
    assert (np.abs(w.astype(np.float64).sum(axis=1) - 1.0) <= 8 * 2.0 ** -24).all()
    assert all(len(set(r)) == 8 for r in ids)


def test_swiglu_vs_torch_float64_and_closed_forms():
    rng = np.random.default_rng(2)
    P, I = 64, 256
    gu = inputs.f32_to_bf16_bits(rng.standard_normal((P, 2 * I)).astype(np.float32) * 3.0)
    h = oracle.swiglu(gu)
    g = torch.from_numpy(inputs.bf16_bits_to_f32(gu[:, :I]).astype(np.float64))
    u = torch.from_numpy(inputs.bf16_bits_to_f32(gu[:, I:]).astype(np.float64))
    ref = (torch.nn.functional.silu(g) * u).to(torch.float32).to(torch.bfloat16)
    ref = ref.view(torch.int16).numpy().view(np.uint16)
    assert _ulp_dist(h, ref).max() <= 1 and (h == ref).mean() > 0.999
    # closed forms: silu(0) = 0; silu(g) -> g for large g; silu(-large) -> 0; gate/up not swapped
    gu = inputs.f32_to_bf16_bits(np.array([[0.0, 64.0, -64.0, 1.0, 3.0, 2.0, 5.0, 0.0]], np.float32))
    h = inputs.bf16_bits_to_f32(oracle.swiglu(gu))[0]
    assert h[0] == 0.0 and h[1] == 128.0 and abs(h[2]) < 1e-20 and h[3] == 0.0
    # silu(1) * 3 with silu(1) = 0.7310585786...
    gu = inputs.f32_to_bf16_bits(np.array([[1.0, 3.0]], np.float32))
    assert inputs.bf16_bits_to_f32(oracle.swiglu(gu))[0, 0] == \
        inputs.bf16_bits_to_f32(inputs.f32_to_bf16_bits(np.array([3 * 0.7310585786300049], np.float32)))[0]


def test_combine_identities():
    rng = np.random.default_rng(3)
    M, k, H, E = 16, 8, 64, 32
    ids, w = inputs.routing(rng, M, E, k)
    row = rng.standard_normal((M, 1, H)).astype(np.float32)
    # 8 identical rows with weights summing to 1 -> that row, within rounding of 8 bf16 terms
    out = oracle.combine(np.repeat(row, k, axis=1).reshape(M * k, H), ids, w)
    got = inputs.bf16_bits_to_f32(out)
    assert np.allclose(got, row[:, 0], rtol=2.0 ** -6, atol=0)
    # k = 1, w = 1: the bf16 rounding of y
    y = rng.standard_normal((M, H)).astype(np.float32)
    out1 = oracle.combine(y, np.zeros((M, 1), np.int32), np.ones((M, 1), np.float32))
    assert np.array_equal(out1, inputs.f32_to_bf16_bits(y))
    # independent of the caller's slot order
    y = rng.standard_normal((M * k, H)).astype(np.float32)
    base = oracle.combine(y, ids, w)
    perm = rng.permutation(k)
    y_p = y.reshape(M, k, H)[:, perm].reshape(M * k, H)
    assert np.array_equal(oracle.combine(y_p, ids[:, perm], w[:, perm]), base)
    # brute force in the stated order
    for t in range(M):
        s = np.zeros(H, np.float32)
        for j in np.argsort(ids[t], kind="stable"):
            c = inputs.bf16_bits_to_f32(inputs.f32_to_bf16_bits(w[t, j] * y[t * k + j]))
            s = (s + c).astype(np.float32)
        assert np.array_equal(base[t], inputs.f32_to_bf16_bits(s))


def _small_case(seed=5, m=24, h=256, i=128, e=8, k=2):
    return inputs.moe_case(seed, m, h=h, i=i, e=e, k=k)


def test_moe_k1_reduces_to_two_linears_and_swiglu():
    c = _small_case(k=1)
    w13c, w13s = oracle.quantize_weight(c.w13)
    w2c, w2s = oracle.quantize_weight(c.w2)
    ones = np.ones_like(c.weights)
    out = oracle.moe(c.x, c.ids, ones, w13c, w13s, w2c, w2s)
    for t in range(c.M):
        e = c.ids[t, 0]
        _, gu = oracle.linear(c.x[t:t + 1], w13c[e], w13s[e])
        h = oracle.swiglu(gu)
        _, y = oracle.linear(h, w2c[e], w2s[e])
        assert np.array_equal(out[t], y[0])


def test_moe_dumps_are_consistent_and_close_to_unquantized_fp64():
    c = _small_case()
    w13c, w13s = oracle.quantize_weight(c.w13)
    w2c, w2s = oracle.quantize_weight(c.w2)
    out, d = oracle.moe(c.x, c.ids, c.weights, w13c, w13s, w2c, w2s, dumps=True)
    assert np.array_equal(d["h"], oracle.swiglu(d["gate_up"]))
    hc, hs = oracle.quantize_act(d["h"])
    assert np.array_equal(hc, d["h_codes"]) and np.array_equal(hs, d["h_scales"])
    assert np.array_equal(out, oracle.combine(d["y32"], c.ids, c.weights))
    # unquantized float64 reference of the whole layer
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
    assert rel < 0.08
    # per-pair gate_up against the dequantized-operand float64 product (tight)
    xc, xs = oracle.quantize_act(c.x)
    xd = DEC[xc] * np.repeat(xs, 128, axis=1)
    for p in range(0, c.M * c.k, 7):
        t, e = p // c.k, c.ids.reshape(-1)[p]
        wd = DEC[w13c[e]] * np.repeat(np.repeat(w13s[e], 128, axis=0), 128, axis=1)
        r = wd @ xd[t]
        g = inputs.bf16_bits_to_f32(d["gate_up"][p]).astype(np.float64)
        assert np.allclose(g, r, rtol=2.0 ** -7, atol=1e-6)


def test_moe_empty_batch_and_empty_experts():
    c = _small_case(m=3, e=8, k=2)
    w13c, w13s = oracle.quantize_weight(c.w13)
    w2c, w2s = oracle.quantize_weight(c.w2)
    out = oracle.moe(c.x, c.ids, c.weights, w13c, w13s, w2c, w2s)      # most experts empty
    assert out.shape == (3, c.H)
    out0 = oracle.moe(c.x[:0], c.ids[:0], c.weights[:0], w13c, w13s, w2c, w2s)
    assert out0.shape == (0, c.H)
