"""GPU parity of the router (bf16 logits GEMM + top-k softmax) and of the o_proj-shaped dense
projection; a live-routed MoE layer end to end."""
import numpy as np
import pytest
import torch

import oracle
from paper_2604_07853_b200 import binding, build, inputs
from util import bits_to_torch, torch_to_bits
from test_gpu_linear import check_linear

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    build.build()
    c = binding.Context(0)
    yield c
    assert c.poll() == 0
    c.close()


def check_router(ctx, seed, m, h, e, k):
    """Logits within the GEMM tolerance of the exact ones; the selection and the weights teacher-forced:
    the oracle's top-k on the GPU's own logits must give the same ids bit for bit (an arg-max decided
    in the same precision on both sides) and weights equal to fp32 rounding (both exp in double)."""
    rng = np.random.default_rng(seed)
    x = inputs.act_bf16(rng, m, h)
    wr = inputs.weight_bf16(rng, e, h)
    logits, ids, wts = ctx.router_fwd(bits_to_torch(x), bits_to_torch(wr), k)
    assert ctx.poll() == 0
    o_logits, _ = oracle.linear_bf16(x, wr)
    nx = np.linalg.norm(inputs.bf16_bits_to_f32(x).astype(np.float64), axis=1)
    nw = np.linalg.norm(inputs.bf16_bits_to_f32(wr).astype(np.float64), axis=1)
    g = logits.cpu().numpy()
    assert (np.abs(g.astype(np.float64) - o_logits) <= 1e-3 * nx[:, None] * nw[None, :]).all()
    o_ids, o_w = oracle.router_topk(g, k)
    assert np.array_equal(ids.cpu().numpy(), o_ids)
    gw = wts.cpu().numpy()
    assert np.allclose(gw, o_w, rtol=2e-7, atol=0.0) and (gw == o_w).mean() > 0.98
    return x, wr, logits, ids, wts


@pytest.mark.parametrize("m,h,e,k", [(1, 64, 8, 1), (5, 256, 16, 4), (300, 2048, 128, 8), (129, 512, 1024, 32),
                                     (64, 128, 40, 8)])
def test_router_shapes(ctx, m, h, e, k):
    check_router(ctx, 400 + m, m, h, e, k)


def test_router_ties_and_equal_logits(ctx):
    """Identical expert rows give identical logits: ties must go to the lower id on the GPU too."""
    rng = np.random.default_rng(3)
    x = inputs.act_bf16(rng, 33, 256)
    wr = inputs.weight_bf16(rng, 16, 256)
    wr[5] = wr[2]
    wr[9] = wr[2]
    wr[15] = wr[0]
    logits, ids, wts = ctx.router_fwd(bits_to_torch(x), bits_to_torch(wr), 6)
    g = logits.cpu().numpy()
    assert np.array_equal(g[:, 5], g[:, 2]) and np.array_equal(g[:, 9], g[:, 2])
    o_ids, o_w = oracle.router_topk(g, 6)
    assert np.array_equal(ids.cpu().numpy(), o_ids)
    zero = torch.zeros((4, 256), dtype=torch.bfloat16, device="cuda")      # all logits equal (0)
    _, ids0, w0 = ctx.router_fwd(zero, bits_to_torch(wr), 4)
    assert ids0.cpu().numpy().tolist() == [[0, 1, 2, 3]] * 4 and torch.all(w0 == 0.25)


def test_routing_does_not_depend_on_the_batch(ctx):
    x, wr, logits, ids, wts = check_router(ctx, 11, 300, 1024, 128, 8)
    xt, wt = bits_to_torch(x), bits_to_torch(wr)
    for rows in ([0], [299], list(range(100, 164))):
        l2, i2, w2 = ctx.router_fwd(xt[rows].contiguous(), wt, 8)
        assert torch.equal(l2, logits[rows]) and torch.equal(i2, ids[rows]) and torch.equal(w2, wts[rows])


@pytest.mark.parametrize("m,h,e,k", [(1, 64, 8, 1), (300, 2048, 128, 8), (1000, 520, 40, 8), (129, 512, 128, 32),
                                     (4133, 1024, 96, 6), (3, 8, 8, 8), (129, 72, 24, 24), (40000, 128, 128, 8)])
def test_one_launch_router_equals_the_two_launch_router(ctx, m, h, e, k):
    """Up to 128 experts the selection runs in the epilogue of the logits GEMM (one launch); the harness
    switch forces the separate selection kernel.  Logits, ids and weights must be the same bytes: the
    same MMA sequence per row, the same selection rule, the softmax summed in the same order."""
    rng = np.random.default_rng(900 + m)
    x = bits_to_torch(inputs.act_bf16(rng, m, h))
    wr_bits = inputs.weight_bf16(rng, e, h)
    wr_bits[e - 1] = wr_bits[0]                              # a tie between the first and the last expert
    wr = bits_to_torch(wr_bits)
    fused = ctx.router_fwd(x, wr, k)
    ctx.harness_set_gemm_path(1)
    split = ctx.router_fwd(x, wr, k)
    ctx.harness_set_gemm_path(0)
    assert ctx.poll() == 0
    for a, b in zip(fused, split):
        assert torch.equal(a.view(torch.int32), b.view(torch.int32))
    ids = fused[1].cpu().numpy()
    assert ((ids >= 0) & (ids < e)).all() and all(len(set(r)) == k for r in ids[:: max(1, m // 50)].tolist())


@pytest.mark.parametrize("e,k,hot", [(128, 16, range(0, 16)), (128, 16, range(16, 32)), (128, 8, range(120, 128)),
                                     (40, 16, range(0, 16)), (128, 16, [0, 17, 33, 34, 35, 50, 66, 67, 82, 98, 99, 100, 113, 114, 126, 127])])
def test_selection_concentrated_in_few_groups(ctx, e, k, hot):
    """The one-launch router keeps one candidate per group of 16 experts and re-scans only the winner's group:
    batches whose k largest logits all sit in one group (also the first, which then runs almost empty) or are
    spread one per group must select what the oracle's plain scan selects on the same logits, in both forms."""
    rng = np.random.default_rng(5 + e + k)
    h = 256
    u = rng.standard_normal(h).astype(np.float32)
    x = (u[None, :] + 0.05 * rng.standard_normal((200, h))).astype(np.float32)
    w = (0.02 * rng.standard_normal((e, h))).astype(np.float32)
    for rank, ex in enumerate(hot):
        w[ex] = (0.2 + 0.01 * ((rank * 7) % len(hot))) * u / np.linalg.norm(u)       # large, distinct, not in id order
    w[hot[1]] = w[hot[0]]                                                            # and one exact tie
    xt = torch.from_numpy(x).to(torch.bfloat16).cuda()
    wt = torch.from_numpy(w).to(torch.bfloat16).cuda()
    fused = ctx.router_fwd(xt, wt, k)
    ctx.harness_set_gemm_path(1)
    split = ctx.router_fwd(xt, wt, k)
    ctx.harness_set_gemm_path(0)
    assert ctx.poll() == 0
    for a, b in zip(fused, split):
        assert torch.equal(a.view(torch.int32), b.view(torch.int32))
    o_ids, _ = oracle.router_topk(fused[0].cpu().numpy(), k)
    ids = fused[1].cpu().numpy()
    assert np.array_equal(ids, o_ids)
    assert set(ids[0, :len(hot)].tolist()) == set(list(hot)[:k]) or len(hot) < k


def test_router_with_non_finite_activations(ctx):
    """Infinite and NaN activations give infinite and NaN logits; whatever the selection does with them, the
    ids stay inside [0, E) and distinct, and both forms of the router do the same."""
    rng = np.random.default_rng(77)
    x = bits_to_torch(inputs.act_bf16(rng, 64, 256)).clone()
    x[3, 5] = float("inf")
    x[7, :] = float("nan")
    x[9, 100] = float("-inf")
    x[11, 1] = float("inf")
    x[11, 2] = float("-inf")
    wr = bits_to_torch(inputs.weight_bf16(rng, 32, 256))
    fused = ctx.router_fwd(x, wr, 4)
    ctx.harness_set_gemm_path(1)
    split = ctx.router_fwd(x, wr, 4)
    ctx.harness_set_gemm_path(0)
    assert ctx.poll() == 0
    ids = fused[1].cpu().numpy()
    assert ((ids >= 0) & (ids < 32)).all() and all(len(set(r)) == 4 for r in ids.tolist())
    assert torch.equal(fused[1], split[1])
    assert torch.equal(fused[0].view(torch.int32), split[0].view(torch.int32))
    assert torch.equal(fused[2].view(torch.int32), split[2].view(torch.int32))
    o_ids, _ = oracle.router_topk(fused[0].cpu().numpy(), 4)
    assert np.array_equal(ids, o_ids)


def test_o_proj_shape(ctx):
    """The attention output projection of the training configuration: K = 4096, N = 2048."""
    check_linear(ctx, inputs.linear_case(21, 200, 2048, 4096))


def test_live_routed_layer_matches_the_oracle_layer(ctx):
    """Router output fed straight into the FP8 MoE layer: same bytes as the oracle's layer run on the
    GPU's routing decision (the layer itself is covered stage by stage elsewhere)."""
    c = inputs.moe_case(12, 64, h=512, i=256, e=16, k=4)
    rng = np.random.default_rng(12)
    wr = inputs.weight_bf16(rng, 16, 512)
    xt = bits_to_torch(c.x)
    _, ids, wts = ctx.router_fwd(xt, bits_to_torch(wr), 4)
    w13c, w13s = ctx.quantize_weight(bits_to_torch(c.w13))
    w2c, w2s = ctx.quantize_weight(bits_to_torch(c.w2))
    out = ctx.moe_fwd(xt, ids, wts, w13c, w13s, w2c, w2s)
    assert ctx.poll() == 0
    ref = oracle.moe(c.x, ids.cpu().numpy(), wts.cpu().numpy(), *(t.cpu().numpy() for t in (w13c, w13s, w2c, w2s)))
    g = inputs.bf16_bits_to_f32(torch_to_bits(out)).astype(np.float64)
    r = inputs.bf16_bits_to_f32(ref).astype(np.float64)
    assert np.linalg.norm(g - r) / np.linalg.norm(r) < 5e-3
