"""GPU parity of the FP4A16 path (Sec. 2.2, floating-point quantization with alpha = 6: e2m1 weights,
bf16 activations): quantizer bit-exact against the oracle, the GEMM and the MoE layer teacher-forced
against the oracle on the GPU's own codes, and the bitwise row invariance across batch shapes."""
import numpy as np
import pytest
import torch

import oracle
from paper_2604_07853_b200 import binding, build, inputs
from test_gpu_w4a16 import DeviceCase, check_linear, check_moe, pack_linear, unpack_lib, unpack_linear
from util import bits_to_torch, torch_to_bits

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    build.build()
    c = binding.Context(0)
    yield c
    assert c.poll() == 0
    c.close()


def host_weights(q):
    """GPU (packed, scales) -> oracle-layout (packed, scales f32 [.., N, K/128])."""
    packed, scales = q
    p = pack_linear(unpack_lib(packed.cpu().numpy()))
    s = inputs.bf16_bits_to_f32(torch_to_bits(scales))
    return p, np.ascontiguousarray(np.swapaxes(s, -1, -2))


class E2m1:
    @staticmethod
    def quantize(ctx, w):
        return ctx.quantize_weight_fp4(w)

    @staticmethod
    def linear(ctx, x, q, **kw):
        return ctx.linear_fwd_fp4a16(x, *q, **kw)

    @staticmethod
    def moe(ctx, x, ids, wts, q13, q2, **kw):
        return ctx.moe_fwd_fp4a16(x, ids, wts, q13, q2, **kw)

    @staticmethod
    def w_hat(q):
        return oracle.dequant_fp4(*host_weights(q))


# ------------------------------------------------------------------------------ quantizer
@pytest.mark.parametrize("e,n,k", [(1, 128, 128), (3, 256, 384), (2, 1536, 2048), (4, 640, 256)])
def test_quantizer_bit_exact(ctx, e, n, k):
    rng = np.random.default_rng(20 + n)
    w = inputs.weight_bf16(rng, e, n, k)
    w[0, 0, :128] = 0                      # an all-zero group
    w[-1, -1, ::3] = 0
    w[0, 1, :128] = 0x8000                 # all negative zero: sign bits are kept
    op, os_ = oracle.quantize_weight_fp4(w)
    gp, gs = host_weights(ctx.quantize_weight_fp4(bits_to_torch(w)))
    assert np.array_equal(unpack_linear(gp), unpack_linear(op))
    assert np.array_equal(gs.view(np.uint32), os_.view(np.uint32))


def test_quantizer_exact_ties_and_saturation(ctx):
    """Multiples of s/4 up to 6 s hit every rounding boundary (.25 .75 1.25 1.75 2.5 3.5 5) exactly, where
    the result must be the neighbour with the even code; several scales, both signs."""
    rng = np.random.default_rng(6)
    w = rng.integers(-24, 25, size=(1, 128, 384)).astype(np.float32) * 0.25      # amax = 6 -> s = 1
    w[:, :, ::128] = 6.0
    w[:, 32:64] *= 8.0
    w[:, 64:96] *= 2.0 ** -10
    w[:, 96:] *= 3.0                       # s = 3: boundaries such as 0.75 = 0.25 s
    wb = inputs.f32_to_bf16_bits(w)
    assert np.array_equal(inputs.bf16_bits_to_f32(wb), w)
    op, os_ = oracle.quantize_weight_fp4(wb)
    assert os_[0, 0, 0] == np.float32(1.0) and os_[0, 100, 0] == np.float32(3.0)
    gp, gs = host_weights(ctx.quantize_weight_fp4(bits_to_torch(wb)))
    assert np.array_equal(unpack_linear(gp), unpack_linear(op))
    assert np.array_equal(gs, os_)
    # every code occurs
    assert set(np.unique(unpack_linear(gp))) == set(range(16))


def test_quantizer_wide_range_of_magnitudes(ctx):
    """Scales from 2^-35 to 2^30: the boundaries b s stay exact and the codes agree everywhere."""
    rng = np.random.default_rng(7)
    w = inputs.bf16_bits_to_f32(inputs.weight_bf16(rng, 1, 128, 1024, std=1.0))
    for g, ex in enumerate([-35, -20, -8, 0, 5, 12, 20, 30]):
        w[:, :, g * 128:(g + 1) * 128] *= np.float32(2.0 ** ex)
    wb = inputs.f32_to_bf16_bits(w)
    op, os_ = oracle.quantize_weight_fp4(wb)
    q = ctx.quantize_weight_fp4(bits_to_torch(wb))
    gp, gs = host_weights(q)
    assert np.array_equal(unpack_linear(gp), unpack_linear(op)) and np.array_equal(gs, os_)
    # and the GEMM's expansion reproduces bf16(s * value) for all of them (identity activations)
    for g in range(8):
        xs = np.zeros((128, 1024), dtype=np.float32)
        xs[np.arange(128), g * 128 + np.arange(128)] = 1.0
        _, y32 = ctx.linear_fwd_fp4a16(bits_to_torch(inputs.f32_to_bf16_bits(xs)), *q, want_f32=True)
        w_hat = inputs.bf16_bits_to_f32(oracle.dequant_fp4(op, os_))[0]
        assert np.array_equal(y32.cpu().numpy(), w_hat[:, g * 128:(g + 1) * 128].T)


def test_quantizer_publish_writes_two_equal_copies(ctx):
    rng = np.random.default_rng(8)
    wt = bits_to_torch(inputs.weight_bf16(rng, 2, 256, 384))
    ref = ctx.quantize_weight_fp4(wt)
    a = tuple(torch.zeros_like(t) for t in ref)
    b = tuple(torch.zeros_like(t) for t in ref)
    ctx.quantize_weight_fp4(wt, out=a, pub=b)
    for r, x, y in zip(ref, a, b):
        assert torch.equal(r, x) and torch.equal(r, y)


# ------------------------------------------------------------------------------ dense GEMM
@pytest.mark.parametrize("m,n,k", [(1, 128, 128), (127, 256, 256), (129, 640, 2048), (300, 1280, 768),
                                   (70, 4096, 2048)])
def test_linear_shapes_and_ragged_tails(ctx, m, n, k):
    check_linear(ctx, 300 + m, m, n, k, fmt=E2m1)


def test_linear_exact_on_representable_data(ctx):
    """Weights that are e2m1 values times a power-of-two scale, integer activations: every product and
    partial sum is exact in fp32, so the GPU must match the exact result bit for bit (a wrong nibble,
    scale, sign or swizzle cannot hide, nor a flushed subnormal: 0.5 is the format's subnormal)."""
    rng = np.random.default_rng(4)
    m, n, k = 37, 256, 384
    x = inputs.f32_to_bf16_bits(rng.integers(-4, 5, size=(m, k)).astype(np.float32))
    table = oracle.e2m1_table().astype(np.float32)
    wf = table[rng.integers(0, 16, size=(n, k))]
    wf[:, ::128] = 6.0                     # amax = 6: s = 1
    wf[n // 2:] *= 0.25                    # s = 1/4
    w = inputs.f32_to_bf16_bits(wf)
    q = ctx.quantize_weight_fp4(bits_to_torch(w))
    assert np.array_equal(inputs.bf16_bits_to_f32(E2m1.w_hat(q)), wf)
    _, y32 = ctx.linear_fwd_fp4a16(bits_to_torch(x), *q, want_f32=True)
    assert np.array_equal(y32.cpu().numpy(), inputs.bf16_bits_to_f32(x) @ wf.T)


def test_linear_rows_do_not_depend_on_the_batch(ctx):
    case = inputs.linear_case(9, 300, 512, 1024)
    q = ctx.quantize_weight_fp4(bits_to_torch(case.w))
    xt = bits_to_torch(case.x)
    full = ctx.linear_fwd_fp4a16(xt, *q)
    for rows in ([0], [299], list(range(120, 140)), list(range(0, 300, 7))):
        part = ctx.linear_fwd_fp4a16(xt[rows].contiguous(), *q)
        assert torch.equal(part, full[rows])


# ------------------------------------------------------------------------------ MoE layer
def test_moe_small_layer(ctx):
    check_moe(ctx, inputs.moe_case(5, 24, h=256, i=128, e=8, k=2), fmt=E2m1)


def test_moe_ragged_groups_and_empty_experts(ctx):
    check_moe(ctx, inputs.moe_case(6, 3, h=256, i=256, e=16, k=4), fmt=E2m1)
    check_moe(ctx, inputs.moe_case(7, 333, h=512, i=256, e=4, k=2), fmt=E2m1)


def test_moe_decode_layer_shape(ctx):
    stats = check_moe(ctx, inputs.config3(), fmt=E2m1)
    assert stats["within1"] > 0.98


def test_moe_rows_do_not_depend_on_the_batch(ctx):
    case = inputs.moe_case(11, 256, h=512, i=256, e=16, k=4, zipf_s=1.1)
    dc = DeviceCase(ctx, case, E2m1)
    full = dc.run(ctx)
    for rows in ([0], [255], list(range(100, 164)), list(range(0, 256, 5))):
        assert torch.equal(dc.run(ctx, rows=rows), full[rows])


def test_argument_checks(ctx):
    dev = torch.device("cuda", 0)
    w = torch.zeros((128, 128), dtype=torch.bfloat16, device=dev)
    q = ctx.quantize_weight_fp4(w)
    with pytest.raises(binding.QarlError):     # N not a multiple of 128
        ctx.quantize_weight_fp4(torch.zeros((64, 128), dtype=torch.bfloat16, device=dev))
    with pytest.raises(binding.QarlError):     # only one of the two published destinations
        ctx._check(ctx.lib.qarl_quantize_weight_fp4(ctx.h, w.data_ptr(), 1, 128, 128, q[0].data_ptr(),
                                                    q[1].data_ptr(), q[0].data_ptr(), None, None))
    assert ctx.poll() == 0
