"""GPU parity: qarl_quantize_weight / qarl_quantize_act are bit-exact against the oracle."""
import numpy as np
import pytest
import torch

import oracle
from paper_2604_07853_b200 import binding, build, inputs
from util import bits_to_torch, to_dev

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    build.build()
    c = binding.Context(0)
    yield c
    assert c.poll() == 0
    c.close()


def _check_act(ctx, x_bits):
    codes, scales = ctx.quantize_act(bits_to_torch(x_bits))
    oc, os_ = oracle.quantize_act(x_bits)
    assert np.array_equal(codes.cpu().numpy(), oc)
    assert np.array_equal(scales.cpu().numpy().view(np.uint32), os_.view(np.uint32))


@pytest.mark.parametrize("m,k", [(16, 512), (1, 128), (3, 2048), (257, 768), (1000, 256)])
def test_quantize_act_bit_exact(ctx, m, k):
    _check_act(ctx, inputs.act_bf16(np.random.default_rng(m * 7 + k), m, k))


def test_quantize_act_every_bf16_value(ctx):
    """Every finite bf16 pattern goes through the cast: groups whose amax is exactly 448 use
    inv = 1, so the code is the e4m3 cast of the bf16 value itself (|v| <= 448), and groups
    with other power-of-two maxima shift the rest of the range onto the grid."""
    allb = np.arange(0, 1 << 16, dtype=np.uint32).astype(np.uint16)
    f = inputs.bf16_bits_to_f32(allb)
    rows = []
    for amax in [448.0, 448.0 * 2.0 ** 20, 448.0 * 2.0 ** -20, 448.0 * 2.0 ** 60, 1.0, 3.0]:
        vals = allb[np.isfinite(f) & (np.abs(f) <= amax)]
        pad = (-len(vals)) % 127
        vals = np.concatenate([vals, np.zeros(pad, np.uint16)]).reshape(-1, 127)
        top = inputs.f32_to_bf16_bits(np.full((vals.shape[0], 1), amax, np.float32))
        rows.append(np.concatenate([top, vals], axis=1))
    x = np.concatenate(rows, axis=0)
    _check_act(ctx, x)


def test_quantize_act_zero_tiny_and_negative_zero(ctx):
    x = np.zeros((4, 256), dtype=np.uint16)
    x[0, 3] = 0x8000
    x[1, 130] = inputs.f32_to_bf16_bits(np.array([1e-30], np.float32))[0]
    x[2, :] = inputs.f32_to_bf16_bits(np.full(256, -2.0 ** -41, np.float32))
    x[3, 5] = 0x0001                                         # smallest bf16 subnormal
    _check_act(ctx, x)


def test_quantize_act_strided_rows(ctx):
    xb = inputs.act_bf16(np.random.default_rng(9), 33, 512)
    xt = bits_to_torch(xb)
    view = xt[:, 128:384]                                   # ldx = 512, K = 256
    codes, scales = ctx.quantize_act(view)
    oc, os_ = oracle.quantize_act(np.ascontiguousarray(xb[:, 128:384]))
    assert np.array_equal(codes.cpu().numpy(), oc)
    assert np.array_equal(scales.cpu().numpy(), os_)


@pytest.mark.parametrize("e,n,k", [(1, 256, 512), (3, 128, 384), (2, 1536, 2048), (1, 5120, 2048)])
def test_quantize_weight_bit_exact(ctx, e, n, k):
    w = inputs.weight_bf16(np.random.default_rng(e + n + k), e, n, k)
    w[0, 5, 7] = 0x8000
    codes, scales = ctx.quantize_weight(bits_to_torch(w))
    oc, os_ = oracle.quantize_weight(w)
    assert np.array_equal(codes.cpu().numpy(), oc)
    assert np.array_equal(scales.cpu().numpy().view(np.uint32), os_.view(np.uint32))


def test_quantize_weight_zero_block_and_2d(ctx):
    w = inputs.weight_bf16(np.random.default_rng(5), 256, 256)
    w[:128, 128:] = 0
    codes, scales = ctx.quantize_weight(bits_to_torch(w))
    oc, os_ = oracle.quantize_weight(w)
    assert codes.shape == (256, 256) and scales.shape == (2, 2)
    assert np.array_equal(codes.cpu().numpy(), oc) and np.array_equal(scales.cpu().numpy(), os_)


def test_empty_and_invalid_arguments(ctx):
    x = torch.zeros((0, 256), dtype=torch.bfloat16, device="cuda")
    c, s = ctx.quantize_act(x)
    assert c.shape == (0, 256)
    with pytest.raises(binding.QarlError) as ei:
        ctx.quantize_act(torch.zeros((4, 100), dtype=torch.bfloat16, device="cuda"))
    assert ei.value.status == -2
    with pytest.raises(binding.QarlError) as ei:
        ctx.quantize_weight(torch.zeros((100, 128), dtype=torch.bfloat16, device="cuda"))
    assert ei.value.status == -2
    xt = torch.zeros((4, 264), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(binding.QarlError) as ei:      # base pointer off by 2 bytes
        ctx.quantize_act(xt[:, 1:257])
    assert ei.value.status == -3
