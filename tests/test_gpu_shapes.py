"""GPU parity on awkward shapes: odd numbers of 128-blocks (half-empty column tiles), the API's
limits on k and E, tiny and single-row groups."""
import numpy as np
import pytest
import torch

import oracle
from paper_2604_07853_b200 import binding, build, inputs
from test_gpu_moe import check_moe
from test_gpu_linear import check_linear

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    build.build()
    c = binding.Context(0)
    yield c
    assert c.poll() == 0
    c.close()


def test_moe_odd_block_counts(ctx):
    # H = 128: the down GEMM's only column tile has an empty second half; I = 384: three gate_up tiles
    check_moe(ctx, inputs.moe_case(21, 70, h=128, i=384, e=4, k=2))
    check_moe(ctx, inputs.moe_case(22, 9, h=384, i=128, e=3, k=3))


def test_moe_topk_and_expert_limits(ctx):
    # k = 32 (the API maximum) of 48 experts; 1024 experts (the API maximum) with most of them empty
    check_moe(ctx, inputs.moe_case(23, 12, h=256, i=128, e=48, k=32), end_to_end=False)
    check_moe(ctx, inputs.moe_case(24, 40, h=128, i=128, e=1024, k=4), end_to_end=False)


def test_moe_single_token_single_expert(ctx):
    check_moe(ctx, inputs.moe_case(25, 1, h=256, i=128, e=8, k=1))
    check_moe(ctx, inputs.moe_case(26, 300, h=256, i=256, e=1, k=1))      # one expert, three row tiles


def test_linear_odd_block_counts_and_long_k(ctx):
    check_linear(ctx, inputs.linear_case(27, 33, 128, 8192))               # 64 K-blocks, one half tile
    check_linear(ctx, inputs.linear_case(28, 513, 896, 384))               # 7 column blocks: last tile half empty


def test_argument_limits_are_rejected(ctx):
    c = inputs.moe_case(29, 4, h=256, i=128, e=8, k=2)
    from util import bits_to_torch, to_dev
    x = bits_to_torch(c.x)
    w13c, w13s = ctx.quantize_weight(bits_to_torch(c.w13))
    w2c, w2s = ctx.quantize_weight(bits_to_torch(c.w2))
    ids = torch.zeros((4, 33), dtype=torch.int32, device="cuda")
    wts = torch.zeros((4, 33), dtype=torch.float32, device="cuda")
    with pytest.raises(binding.QarlError) as ei:
        ctx.moe_fwd(x, ids, wts, w13c, w13s, w2c, w2s)                     # k = 33 > 32
    assert ei.value.status == -1


def test_argument_limits_of_the_widened_entry_points(ctx):
    """Bad shapes come back as status codes before anything is launched."""
    bf = lambda *s: torch.zeros(s, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(binding.QarlError) as ei:
        ctx.quantize_weight_w4(bf(1, 100, 128))                 # N % 128 != 0
    assert ei.value.status == -2
    with pytest.raises(binding.QarlError) as ei:
        ctx.quantize_weight_w4(bf(1, 128, 192))                 # K % 128 != 0
    assert ei.value.status == -2
    with pytest.raises(binding.QarlError) as ei:
        ctx.linear_bwd(bf(4, 12), bf(4, 16), bf(12, 16))         # N % 8 != 0
    assert ei.value.status == -2
    f32 = lambda *s: torch.zeros(s, dtype=torch.float32, device="cuda")
    off = torch.tensor([0, 4], dtype=torch.int64, device="cuda")
    with pytest.raises(binding.QarlError) as ei:
        ctx.tbpo_loss(f32(4), f32(4), f32(4), off, f32(1), cap=1.0)   # the cap must exceed 1
    assert ei.value.status == -1
    with pytest.raises(binding.QarlError) as ei:
        ctx.router_fwd(bf(4, 64), bf(8, 64), 9)                  # k > E
    assert ei.value.status == -1
    with pytest.raises(binding.QarlError) as ei:
        ctx.router_fwd(bf(4, 64), bf(1032, 64), 8)               # E > 1024
    assert ei.value.status == -2
    assert ctx.poll() == 0
