"""GPU parity of the straight-through backward (Sec. 3.1 item 2): dX = dY W, dW = dY^T X on bf16
masters against the oracle; exact on integer data; rows of dX independent of the batch."""
import numpy as np
import pytest
import torch

import oracle
from paper_2604_07853_b200 import binding, build, inputs
from util import bf16_ulp_dist, bits_to_torch, torch_to_bits

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    build.build()
    c = binding.Context(0)
    yield c
    assert c.poll() == 0
    c.close()


def _case(seed, m, n, k):
    rng = np.random.default_rng(seed)
    return inputs.act_bf16(rng, m, n), inputs.act_bf16(rng, m, k), inputs.weight_bf16(rng, n, k)


def _norms(a_bits, axis):
    return np.linalg.norm(inputs.bf16_bits_to_f32(a_bits).astype(np.float64), axis=axis)


def check_bwd(ctx, seed, m, n, k):
    """fp32: |gpu - oracle| <= 1e-3 * ||row of A|| * ||row of B|| (the oracle sums exactly; the
    tensor core adds exact products in fp32).  dX bf16 = rounding of the GPU's fp32, bit for bit."""
    dy, x, w = _case(seed, m, n, k)
    dx16, dx32, dw32 = ctx.linear_bwd(bits_to_torch(dy), bits_to_torch(x), bits_to_torch(w), want_dx_f32=True)
    assert ctx.poll() == 0
    o_dx32, o_dx16, o_dw32 = oracle.linear_bwd(dy, x, w)
    tol_dx = 1e-3 * _norms(dy, 1)[:, None] * _norms(w, 0)[None, :]
    err = np.abs(dx32.cpu().numpy().astype(np.float64) - o_dx32)
    assert (err <= tol_dx).all(), f"dX max err/tol {(err / tol_dx).max()}"
    g16 = torch_to_bits(dx16)
    assert np.array_equal(g16, oracle.bf16_rne(dx32.cpu().numpy()))
    assert (bf16_ulp_dist(g16, o_dx16) > 1).mean() < 1e-3
    tol_dw = 1e-3 * _norms(dy, 0)[:, None] * _norms(x, 0)[None, :]
    err = np.abs(dw32.cpu().numpy().astype(np.float64) - o_dw32)
    assert (err <= tol_dw).all(), f"dW max err/tol {(err / tol_dw).max()}"


@pytest.mark.parametrize("m,n,k", [(1, 8, 8), (64, 128, 128), (127, 256, 256), (129, 520, 264), (300, 1280, 768),
                                   (1000, 136, 2048), (257, 2048, 72)])
def test_shapes_and_ragged_edges(ctx, m, n, k):
    check_bwd(ctx, 300 + m, m, n, k)


def test_exact_on_integer_data(ctx):
    """Every product and partial sum is exact in fp32: a wrong operand orientation, swizzle or
    descriptor stride cannot hide behind a tolerance."""
    rng = np.random.default_rng(6)
    m, n, k = 200, 264, 392
    dy = inputs.f32_to_bf16_bits(rng.integers(-4, 5, size=(m, n)).astype(np.float32))
    x = inputs.f32_to_bf16_bits(rng.integers(-4, 5, size=(m, k)).astype(np.float32))
    w = inputs.f32_to_bf16_bits(rng.integers(-4, 5, size=(n, k)).astype(np.float32))
    _, dx32, dw32 = ctx.linear_bwd(bits_to_torch(dy), bits_to_torch(x), bits_to_torch(w), want_dx_f32=True)
    dyf, xf, wf = (inputs.bf16_bits_to_f32(a) for a in (dy, x, w))
    assert np.array_equal(dx32.cpu().numpy(), dyf @ wf)
    assert np.array_equal(dw32.cpu().numpy(), dyf.T @ xf)


def test_dx_rows_do_not_depend_on_the_batch(ctx):
    dy, x, w = _case(7, 300, 512, 1024)
    dyt, xt, wt = bits_to_torch(dy), bits_to_torch(x), bits_to_torch(w)
    full, _, _ = ctx.linear_bwd(dyt, xt, wt, dw=False)
    for rows in ([0], [299], list(range(120, 140)), list(range(0, 300, 7))):
        part, _, _ = ctx.linear_bwd(dyt[rows].contiguous(), xt[rows].contiguous(), wt, dw=False)
        assert torch.equal(part, full[rows])


def test_qkv_projection_shape_sampled(ctx):
    """K = 2048, N = 5120, M = 8192 (the dense projection of the training configuration): sampled
    rows of dX and of dW against the oracle."""
    dy, x, w = _case(8, 8192, 5120, 2048)
    dyt, xt, wt = bits_to_torch(dy), bits_to_torch(x), bits_to_torch(w)
    dx16, dx32, dw32 = ctx.linear_bwd(dyt, xt, wt, want_dx_f32=True)
    assert ctx.poll() == 0
    rows = np.array([0, 127, 128, 4095, 8191] + list(np.random.default_rng(1).integers(0, 8192, 11)))
    o_dx32, _, _ = oracle.linear_bwd(dy[rows], x[rows], w)
    tol = 1e-3 * _norms(dy[rows], 1)[:, None] * _norms(w, 0)[None, :]
    g = dx32[torch.from_numpy(rows).cuda()].cpu().numpy().astype(np.float64)
    assert (np.abs(g - o_dx32) <= tol).all()
    # dW rows n: needs the full token dimension; take a few output features
    feats = np.array([0, 1, 255, 256, 5119, 2500])
    _, _, o_dw = oracle.linear_bwd(np.ascontiguousarray(dy[:, feats]), x, w[feats])
    tol = 1e-3 * _norms(dy[:, feats], 0)[:, None] * _norms(x, 0)[None, :]
    g = dw32[torch.from_numpy(feats).cuda()].cpu().numpy().astype(np.float64)
    assert (np.abs(g - o_dw) <= tol).all()


def test_quantize_weight_publish_writes_two_equal_copies(ctx):
    """Sec. 3.1 item 3: the published tensors are the ones the training forward uses, bit for bit."""
    rng = np.random.default_rng(9)
    w = inputs.weight_bf16(rng, 3, 256, 384)
    wt = bits_to_torch(w)
    codes, scales = ctx.quantize_weight(wt)
    c1, s1 = torch.zeros_like(codes), torch.zeros_like(scales)
    c2, s2 = torch.zeros_like(codes), torch.zeros_like(scales)
    ctx.quantize_weight_publish(wt, c1, s1, c2, s2)
    assert torch.equal(c1, codes) and torch.equal(c2, codes)
    assert torch.equal(s1, scales) and torch.equal(s2, scales)
    oc, os_ = oracle.quantize_weight(w)
    assert np.array_equal(c2.cpu().numpy(), oc) and np.array_equal(s2.cpu().numpy(), os_)
