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
