"""GPU parity: qarl_linear_fwd / qarl_linear_fwd_q against the oracle, and row invariance."""
import numpy as np
import pytest
import torch

import oracle
from paper_2604_07853_b200 import binding, build, inputs
from util import bf16_ulp_dist, bits_to_torch, to_dev, torch_to_bits

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    build.build()
    c = binding.Context(0)
    yield c
    assert c.poll() == 0
    c.close()


def _dequant_norms(xc, xs, wc, ws):
    dec = oracle.e4m3_decode_table()
    xd = dec[xc] * np.repeat(xs.astype(np.float64), 128, axis=1)
    wd = dec[wc] * np.repeat(np.repeat(ws.astype(np.float64), 128, axis=0), 128, axis=1)
    return np.linalg.norm(xd, axis=1), np.linalg.norm(wd, axis=1)


def check_linear(ctx, case, via_q=False):
    """Teacher-forced: the oracle consumes the GPU's own codes and scales, so only the GEMM is
    under test.  fp32: |gpu - oracle| <= 1e-3 * ||x^_row|| * ||w^_col||.  bf16: equal to the
    rounding of the GPU's fp32 bit for bit, and within 1 ulp of the oracle's bf16 except where
    cancellation makes 1 ulp smaller than the fp32 bound (counted, must be rare)."""
    wt = bits_to_torch(case.w)
    wc, ws = ctx.quantize_weight(wt)
    xt = bits_to_torch(case.x)
    xc, xs = ctx.quantize_act(xt)
    if via_q:
        y, y32 = ctx.linear_fwd_q(xc, xs, wc, ws, want_f32=True)
    else:
        y, y32 = ctx.linear_fwd(xt, wc, ws, want_f32=True)
    assert ctx.poll() == 0
    xc_h, xs_h, wc_h, ws_h = (t.cpu().numpy() for t in (xc, xs, wc, ws))
    o32, o16 = oracle.linear_q(xc_h, xs_h, wc_h, ws_h)
    g32 = y32.cpu().numpy()
    g16 = torch_to_bits(y)
    nx, nw = _dequant_norms(xc_h, xs_h, wc_h, ws_h)
    tol = 1e-3 * nx[:, None] * nw[None, :]
    err = np.abs(g32.astype(np.float64) - o32.astype(np.float64))
    assert (err <= tol).all(), f"max err/tol = {(err / tol).max()}"
    assert np.array_equal(g16, oracle.bf16_rne(g32))
    d = bf16_ulp_dist(g16, o16)
    far = d > 1
    assert (err[far] <= tol[far]).all()
    assert far.mean() < 1e-3, f"{far.sum()} elements beyond 1 ulp"
    return dict(max_rel=float((err / tol).max()), exact=float((d == 0).mean()))


def test_config1(ctx):
    stats = check_linear(ctx, inputs.config1())
    assert stats["exact"] > 0.95


@pytest.mark.parametrize("m,n,k", [(1, 128, 128), (127, 256, 256), (128, 384, 512), (129, 640, 2048),
                                   (300, 1280, 768), (5, 256, 4096)])
def test_shapes_and_ragged_tails(ctx, m, n, k):
    check_linear(ctx, inputs.linear_case(100 + m, m, n, k))


def test_prequantized_entry_point_matches(ctx):
    case = inputs.linear_case(7, 70, 512, 512)
    check_linear(ctx, case, via_q=True)
    wt, xt = bits_to_torch(case.w), bits_to_torch(case.x)
    wc, ws = ctx.quantize_weight(wt)
    xc, xs = ctx.quantize_act(xt)
    a = ctx.linear_fwd(xt, wc, ws)
    b = ctx.linear_fwd_q(xc, xs, wc, ws)
    assert torch.equal(a, b)


def test_exact_special_case_bitwise_equal_to_fp64_product(ctx):
    """Lossless quantization and integer partial sums below 2^24: GPU == oracle == the fp64
    product of the original tensors, whatever order the tensor core adds in."""
    rng = np.random.default_rng(1)
    M, N, K = 150, 256, 512
    x = rng.integers(-8, 9, size=(M, K)).astype(np.float64)
    w = rng.integers(-8, 9, size=(N, K)).astype(np.float64)
    x[:, ::128] = 448.0
    w[3, ::128] = -448.0
    w[200, ::128] = 448.0
    x *= 2.0 ** -3
    w *= 2.0 ** 2
    xb, wb = inputs.f32_to_bf16_bits(x), inputs.f32_to_bf16_bits(w)
    wc, ws = ctx.quantize_weight(bits_to_torch(wb))
    y, y32 = ctx.linear_fwd(bits_to_torch(xb), wc, ws, want_f32=True)
    assert np.array_equal(y32.cpu().numpy().astype(np.float64), x @ w.T)
    o32, o16 = oracle.linear(xb, wc.cpu().numpy(), ws.cpu().numpy())
    assert np.array_equal(y32.cpu().numpy(), o32) and np.array_equal(torch_to_bits(y), o16)


def test_row_invariance_across_batch_size_and_position(ctx):
    """App. C: a row's output bytes do not depend on M, on its position or on its neighbours."""
    case = inputs.linear_case(21, 300, 512, 1024)
    wc, ws = ctx.quantize_weight(bits_to_torch(case.w))
    xt = bits_to_torch(case.x)
    full = ctx.linear_fwd(xt, wc, ws).clone()
    rng = np.random.default_rng(0)
    for m in (1, 8, 64, 129, 256):
        idx = torch.from_numpy(rng.permutation(300)[:m].copy()).cuda()
        sub = ctx.linear_fwd(xt[idx].contiguous(), wc, ws)
        assert torch.equal(sub, full[idx]), m
    again = ctx.linear_fwd(xt, wc, ws)
    assert torch.equal(again, full)


def test_config2_decode_shape(ctx):
    check_linear(ctx, inputs.config2(64))


def test_linear_empty_and_errors(ctx):
    case = inputs.linear_case(3, 4, 128, 128)
    wc, ws = ctx.quantize_weight(bits_to_torch(case.w))
    y = ctx.linear_fwd(torch.zeros((0, 128), dtype=torch.bfloat16, device="cuda"), wc, ws)
    assert y.shape == (0, 128)
    lib = ctx.lib
    x = bits_to_torch(case.x)
    out = torch.empty((4, 128), dtype=torch.bfloat16, device="cuda")
    wsb = torch.empty(256, dtype=torch.uint8, device="cuda")
    rc = lib.qarl_linear_fwd(ctx.h, x.data_ptr(), 4, 128, wc.data_ptr(), ws.data_ptr(), 128, out.data_ptr(),
                             None, wsb.data_ptr(), 16, None)
    assert rc == -4                                           # workspace too small
    rc = lib.qarl_linear_fwd(ctx.h, None, 4, 128, wc.data_ptr(), ws.data_ptr(), 128, out.data_ptr(),
                             None, wsb.data_ptr(), 4096, None)
    assert rc == -1
