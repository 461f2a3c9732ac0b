"""Pins for the oracle's straight-through backward of the linear layer (Sec. 3.1 item 2:
low-bit forward, full-precision backward on the bf16 master weights)."""
import numpy as np

import oracle
from paper_2604_07853_b200 import inputs


def _ints(rng, shape, lo=-6, hi=7):
    return inputs.f32_to_bf16_bits(rng.integers(lo, hi, size=shape).astype(np.float32))


def test_hand_worked_2x2():
    """y = x W^T with W = [[1, 2], [3, 4]], x = [[1, -1]], dY = [[2, 5]]:
    dX = dY W = [2*1 + 5*3, 2*2 + 5*4] = [17, 24];  dW = dY^T x = [[2, -2], [5, -5]]."""
    # embed in the smallest shapes the layout allows (any M, N, K is accepted by the oracle)
    w = inputs.f32_to_bf16_bits(np.array([[1, 2], [3, 4]], np.float32))
    x = inputs.f32_to_bf16_bits(np.array([[1, -1]], np.float32))
    dy = inputs.f32_to_bf16_bits(np.array([[2, 5]], np.float32))
    dx32, dx16, dw32 = oracle.linear_bwd(dy, x, w)
    assert np.array_equal(dx32, [[17, 24]]) and np.array_equal(dw32, [[2, -2], [5, -5]])
    assert np.array_equal(inputs.bf16_bits_to_f32(dx16), dx32)


def test_adjoint_identity_exact_on_integers():
    """<dY, X W^T> = <dX, X> = <dW, W>: the defining property of the two gradients, checked with
    integer data where every quantity is exact.  A transposed operand or a swapped index in either
    gradient breaks one of the two equalities."""
    rng = np.random.default_rng(0)
    M, N, K = 13, 7, 11
    x, w, dy = _ints(rng, (M, K)), _ints(rng, (N, K)), _ints(rng, (M, N))
    xf, wf, dyf = (inputs.bf16_bits_to_f32(a).astype(np.int64) for a in (x, w, dy))
    y32, _ = oracle.linear_bf16(x, w)                 # the forward the gradients belong to
    dx32, _, dw32 = oracle.linear_bwd(dy, x, w)
    lhs = int((dyf * y32.astype(np.int64)).sum())
    assert lhs == int((dx32.astype(np.int64) * xf).sum()) == int((dw32.astype(np.int64) * wf).sum())


def test_special_cases():
    rng = np.random.default_rng(1)
    M, K = 9, 16
    x, dy = _ints(rng, (M, K)), _ints(rng, (M, K))
    eye = inputs.f32_to_bf16_bits(np.eye(K, dtype=np.float32))
    dx32, _, dw32 = oracle.linear_bwd(dy, x, eye)     # W = I: dX = dY
    assert np.array_equal(dx32, inputs.bf16_bits_to_f32(dy))
    # one sample (M = 1): dW is the outer product dy^T x
    dx32, _, dw32 = oracle.linear_bwd(dy[:1], x[:1], eye)
    assert np.array_equal(dw32, np.outer(inputs.bf16_bits_to_f32(dy[0]), inputs.bf16_bits_to_f32(x[0])))
    # rows are independent in dX, samples add up in dW
    a = oracle.linear_bwd(dy[:4], x[:4], eye)
    b = oracle.linear_bwd(dy[4:], x[4:], eye)
    full = oracle.linear_bwd(dy, x, eye)
    assert np.array_equal(np.concatenate([a[0], b[0]]), full[0]) and np.array_equal(a[2] + b[2], full[2])


def test_finite_difference_of_the_forward():
    """d/dX and d/dW of L = sum(dY * (X W^T)) by central differences on the (linear) forward."""
    rng = np.random.default_rng(2)
    M, N, K = 5, 6, 8
    x, w, dy = _ints(rng, (M, K)), _ints(rng, (N, K)), _ints(rng, (M, N))
    xf, wf, dyf = (inputs.bf16_bits_to_f32(a).astype(np.float64) for a in (x, w, dy))
    dx32, _, dw32 = oracle.linear_bwd(dy, x, w)
    L = lambda X, W: float((dyf * (X @ W.T)).sum())
    for (i, j) in [(0, 0), (2, 5), (4, 7)]:
        e = np.zeros_like(xf); e[i, j] = 1.0
        assert (L(xf + e, wf) - L(xf - e, wf)) / 2 == dx32[i, j]
    for (i, j) in [(0, 0), (3, 4), (5, 7)]:
        e = np.zeros_like(wf); e[i, j] = 1.0
        assert (L(xf, wf + e) - L(xf, wf - e)) / 2 == dw32[i, j]


def test_rounding_is_one_rounding_of_the_exact_sum():
    rng = np.random.default_rng(3)
    x = inputs.act_bf16(rng, 40, 128)
    w = inputs.weight_bf16(rng, 24, 128)
    dy = inputs.act_bf16(rng, 40, 24)
    dx32, dx16, dw32 = oracle.linear_bwd(dy, x, w)
    xf, wf, dyf = (inputs.bf16_bits_to_f32(a).astype(np.float64) for a in (x, w, dy))
    assert np.array_equal(dx32, (dyf @ wf).astype(np.float32))
    assert np.array_equal(dw32, (dyf.T @ xf).astype(np.float32))
    assert np.array_equal(dx16, inputs.f32_to_bf16_bits(dx32))


def test_grouped_backward_is_the_per_expert_backward():
    """Adjoint identity per expert on integers, an empty expert, and E = 1 equals the dense call."""
    rng = np.random.default_rng(4)
    E, N, K = 4, 6, 5
    off = np.array([0, 3, 3, 10, 12])
    P = off[-1]
    x, dy, w = _ints(rng, (P, K)), _ints(rng, (P, N)), _ints(rng, (E, N, K))
    dx32, dx16, dw32 = oracle.grouped_linear_bwd(dy, x, w, off)
    assert (dw32[1] == 0).all()
    xf, dyf, wf = (inputs.bf16_bits_to_f32(a).astype(np.int64) for a in (x, dy, w))
    for e in range(E):
        a, b = off[e], off[e + 1]
        y = xf[a:b] @ wf[e].T
        lhs = int((dyf[a:b] * y).sum())
        assert lhs == int((dx32[a:b].astype(np.int64) * xf[a:b]).sum()) == int((dw32[e].astype(np.int64) * wf[e]).sum())
    d1 = oracle.grouped_linear_bwd(dy, x, w[:1], np.array([0, P]))
    d0 = oracle.linear_bwd(dy, x, w[0])
    assert np.array_equal(d1[0], d0[0]) and np.array_equal(d1[2][0], d0[2])


def _layer_f64(x, w13, w2, ids, wts):
    """The layer as a smooth function in float64 (no quantization, no rounding): the function whose
    derivative the straight-through backward approximates."""
    M, k = ids.shape
    I = w2.shape[2]
    out = np.zeros((M, w2.shape[1]))
    for t in range(M):
        for j in range(k):
            e = ids[t, j]
            gu = w13[e] @ x[t]
            g, u = gu[:I], gu[I:]
            out[t] += wts[t, j] * (w2[e] @ (g / (1 + np.exp(-g)) * u))
    return out


def test_swiglu_bwd_is_the_derivative_of_swiglu():
    rng = np.random.default_rng(5)
    g = rng.normal(0, 1.5, size=(4, 16))
    u = rng.normal(0, 1.0, size=(4, 16))
    gu = inputs.f32_to_bf16_bits(np.concatenate([g, u], axis=1).astype(np.float32))
    ones = inputs.f32_to_bf16_bits(np.ones((4, 16), np.float32))
    d = inputs.bf16_bits_to_f32(oracle.swiglu_bwd(gu, ones)).astype(np.float64)
    gq = inputs.bf16_bits_to_f32(gu).astype(np.float64)
    gg, uu = gq[:, :16], gq[:, 16:]
    f = lambda a, b: a / (1 + np.exp(-a)) * b
    eps = 1e-6
    assert np.allclose(d[:, :16], (f(gg + eps, uu) - f(gg - eps, uu)) / (2 * eps), rtol=1e-2, atol=1e-3)   # bf16 output
    assert np.allclose(d[:, 16:], (f(gg, uu + eps) - f(gg, uu - eps)) / (2 * eps), rtol=1e-2, atol=1e-3)
    # g = 0: silu'(0) = 1/2, silu(0) = 0
    z = inputs.f32_to_bf16_bits(np.array([[0.0, 2.0]], np.float32))
    out = inputs.bf16_bits_to_f32(oracle.swiglu_bwd(z, inputs.f32_to_bf16_bits(np.array([[3.0]], np.float32))))
    assert out.tolist() == [[3.0, 0.0]]


def test_layer_backward_against_numeric_derivatives_of_the_smooth_layer():
    """L = <dOut, layer(x, W13, W2)>: central differences of the float64 layer w.r.t. entries of x, W13,
    W2 and the routing weights against the oracle's backward (which rounds intermediates to bf16 and
    uses the forward's saved activations): agreement to a few percent pins every index, transpose,
    sign and the sorted-order bookkeeping."""
    c = inputs.moe_case(31, 10, h=128, i=128, e=4, k=2)
    rng = np.random.default_rng(31)
    x = inputs.bf16_bits_to_f32(c.x).astype(np.float64)
    w13 = inputs.bf16_bits_to_f32(c.w13).astype(np.float64)
    w2 = inputs.bf16_bits_to_f32(c.w2).astype(np.float64)
    wts = c.weights.astype(np.float64)
    dout_bits = inputs.f32_to_bf16_bits(rng.normal(0, 1, size=(c.M, c.H)).astype(np.float32))
    dout = inputs.bf16_bits_to_f32(dout_bits).astype(np.float64)
    # saved activations of a forward in bf16 on the masters (what the backward is given), sorted order
    off, srt, _ = oracle.permute(c.ids, c.E)
    tok, exp = srt // c.k, c.ids.reshape(-1)[srt]
    gu = np.stack([w13[e] @ x[t] for t, e in zip(tok, exp)])
    gu_bits = inputs.f32_to_bf16_bits(gu.astype(np.float32))
    h_bits = oracle.swiglu(gu_bits)
    y32 = np.stack([w2[e] @ inputs.bf16_bits_to_f32(h_bits[q]).astype(np.float64) for q, e in enumerate(exp)]).astype(np.float32)
    out = oracle.moe_bwd(c.x, c.ids, c.weights, c.w13, c.w2, gu_bits, h_bits, dout_bits, y32=y32)
    L = lambda X, A, B, Wt: float((dout * _layer_f64(X, A, B, c.ids, Wt)).sum())
    dx = inputs.bf16_bits_to_f32(out["dx"]).astype(np.float64)
    scale = np.abs(dx).mean()

    def close(num, got, ref_scale):
        return abs(num - got) <= 0.03 * abs(num) + 0.02 * ref_scale

    eps = 1e-4
    for (t, hh) in [(0, 0), (3, 77), (9, 127), (5, 64)]:
        e_ = np.zeros_like(x); e_[t, hh] = eps
        num = (L(x + e_, w13, w2, wts) - L(x - e_, w13, w2, wts)) / (2 * eps)
        assert close(num, dx[t, hh], scale), (t, hh, num, dx[t, hh])
    used = np.unique(c.ids)
    for e in used[:3]:
        for (n, hh) in [(0, 0), (130, 5), (255, 127)]:
            e_ = np.zeros_like(w13); e_[e, n, hh] = eps
            num = (L(x, w13 + e_, w2, wts) - L(x, w13 - e_, w2, wts)) / (2 * eps)
            assert close(num, out["dw13"][e, n, hh], np.abs(out["dw13"][e]).mean()), (e, n, hh)
        for (hh, i) in [(0, 0), (100, 127), (64, 3)]:
            e_ = np.zeros_like(w2); e_[e, hh, i] = eps
            num = (L(x, w13, w2 + e_, wts) - L(x, w13, w2 - e_, wts)) / (2 * eps)
            assert close(num, out["dw2"][e, hh, i], np.abs(out["dw2"][e]).mean()), (e, hh, i)
    for (t, j) in [(0, 0), (4, 1), (9, 0)]:
        e_ = np.zeros_like(wts); e_[t, j] = eps
        num = (L(x, w13, w2, wts + e_) - L(x, w13, w2, wts - e_)) / (2 * eps)
        assert close(num, out["dwts"][t, j], np.abs(out["dwts"]).mean()), (t, j)
    # an expert no token chose has zero weight gradients
    for e in set(range(c.E)) - set(used.tolist()):
        assert (out["dw13"][e] == 0).all() and (out["dw2"][e] == 0).all()
