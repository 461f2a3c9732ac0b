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


# ------------------------------------------------------------------------------ grouped (expert) backward
def check_grouped(ctx, seed, sizes, n, k, exact=False):
    rng = np.random.default_rng(seed)
    E = len(sizes)
    off = np.concatenate([[0], np.cumsum(sizes)]).astype(np.int32)
    P = int(off[-1])
    if exact:
        mk = lambda *s: inputs.f32_to_bf16_bits(rng.integers(-4, 5, size=s).astype(np.float32))
        dy, x, w = mk(P, n), mk(P, k), mk(E, n, k)
    else:
        dy, x = inputs.act_bf16(rng, P, n), inputs.act_bf16(rng, P, k)
        w = inputs.weight_bf16(rng, E, n, k)
    dx16, dx32, dw32 = ctx.grouped_linear_bwd(bits_to_torch(dy), bits_to_torch(x), bits_to_torch(w),
                                              torch.from_numpy(off).cuda(), want_dx_f32=True)
    assert ctx.poll() == 0
    o_dx32, o_dx16, o_dw32 = oracle.grouped_linear_bwd(dy, x, w, off)
    g_dx, g_dw = dx32.cpu().numpy(), dw32.cpu().numpy()
    if exact:
        assert np.array_equal(g_dx, o_dx32) and np.array_equal(g_dw, o_dw32)
        return
    for e in range(E):
        a, b = off[e], off[e + 1]
        tol = 1e-3 * _norms(dy[a:b], 1)[:, None] * _norms(w[e], 0)[None, :]
        assert (np.abs(g_dx[a:b].astype(np.float64) - o_dx32[a:b]) <= tol).all()
        tol = 1e-3 * _norms(dy[a:b], 0)[:, None] * _norms(x[a:b], 0)[None, :] if b > a else np.zeros((n, k))
        assert (np.abs(g_dw[e].astype(np.float64) - o_dw32[e]) <= tol).all(), f"expert {e}"
    assert np.array_equal(torch_to_bits(dx16), oracle.bf16_rne(g_dx))


def test_grouped_exact_on_integer_data(ctx):
    """Ragged groups around the 64-row step and the 128-row tile, empty experts first, last and in the
    middle: every value exact, so one row leaking from a neighbouring expert cannot hide."""
    check_grouped(ctx, 1, [0, 1, 63, 64, 65, 0, 127, 128, 129, 200, 0], 128, 264, exact=True)
    check_grouped(ctx, 2, [5], 64, 8, exact=True)
    check_grouped(ctx, 3, [0, 0, 7, 0], 192, 512, exact=True)


def test_grouped_random_data(ctx):
    check_grouped(ctx, 4, [300, 17, 0, 1000, 64, 129], 256, 512)


def test_grouped_expert_projection_shapes(ctx):
    """The two expert projections of the layer at a reduced expert count: down (N = 2048 -> K = 768)
    and gate_up (N = 1536 -> K = 2048), Zipf-like group sizes."""
    sizes = [900, 40, 333, 0, 128, 1, 77, 569]
    check_grouped(ctx, 5, sizes, 2048, 768)
    check_grouped(ctx, 6, sizes, 1536, 2048)


# ------------------------------------------------------------------------------ MoE layer backward
def check_moe_bwd(ctx, case, seed):
    """FP8 forward on the GPU (saving gate_up, h and the fp32 down output), then the backward; the
    oracle's backward runs on the same saved tensors.  Intermediates cross op boundaries in bf16 on
    both sides and may differ by one bf16 step where the GPU's fp32 accumulation order rounds the
    other way, so the end-to-end bars are norms: 1 % on dx and the weight gradients per expert,
    1e-4 on the routing-weight gradient (a plain fp32 dot product)."""
    from util import to_dev
    c = case
    rng = np.random.default_rng(seed)
    dout = inputs.f32_to_bf16_bits(rng.normal(0, 1, size=(c.M, c.H)).astype(np.float32))
    xt, ids, wts = bits_to_torch(c.x), to_dev(c.ids), to_dev(c.weights)
    w13t, w2t = bits_to_torch(c.w13), bits_to_torch(c.w2)
    w13c, w13s = ctx.quantize_weight(w13t)
    w2c, w2s = ctx.quantize_weight(w2t)
    _, d = ctx.moe_fwd(xt, ids, wts, w13c, w13s, w2c, w2s, debug=True)
    out = ctx.moe_bwd(xt, ids, wts, w13t, w2t, d["gate_up"], d["h"], bits_to_torch(dout), down_f32=d["down_f32"])
    assert ctx.poll() == 0
    ref = oracle.moe_bwd(c.x, c.ids, c.weights, c.w13, c.w2, torch_to_bits(d["gate_up"]), torch_to_bits(d["h"]), dout,
                         y32=d["down_f32"].cpu().numpy())
    rel = lambda g, r: np.linalg.norm(g.astype(np.float64) - r.astype(np.float64)) / max(np.linalg.norm(r.astype(np.float64)), 1e-30)
    gdx = inputs.bf16_bits_to_f32(torch_to_bits(out["dx"]))
    assert rel(gdx, inputs.bf16_bits_to_f32(ref["dx"])) < 1e-2
    g13, g2 = out["dw13"].cpu().numpy(), out["dw2"].cpu().numpy()
    sizes = np.diff(ref["offsets"])
    for e in range(c.E):
        if sizes[e] == 0:
            assert (g13[e] == 0).all() and (g2[e] == 0).all()
        else:
            assert rel(g13[e], ref["dw13"][e]) < 1e-2 and rel(g2[e], ref["dw2"][e]) < 1e-2, e
    assert rel(out["dwts"].cpu().numpy(), ref["dwts"]) < 1e-4
    return out, ref


def test_moe_layer_backward_small(ctx):
    check_moe_bwd(ctx, inputs.moe_case(41, 24, h=256, i=128, e=8, k=2), 41)


def test_moe_layer_backward_ragged_and_empty_experts(ctx):
    check_moe_bwd(ctx, inputs.moe_case(42, 3, h=256, i=256, e=16, k=4), 42)
    check_moe_bwd(ctx, inputs.moe_case(43, 333, h=512, i=256, e=4, k=2), 43)


def test_moe_layer_backward_skewed(ctx):
    check_moe_bwd(ctx, inputs.moe_case(44, 600, h=256, i=128, e=32, k=8, zipf_s=1.1), 44)


def test_moe_layer_backward_token_rows_do_not_depend_on_the_batch(ctx):
    """dx of a token depends only on that token (weight gradients of course add over the batch)."""
    from util import to_dev
    c = inputs.moe_case(45, 128, h=256, i=128, e=8, k=2)
    rng = np.random.default_rng(45)
    dout = bits_to_torch(inputs.f32_to_bf16_bits(rng.normal(0, 1, size=(c.M, c.H)).astype(np.float32)))
    xt, ids, wts = bits_to_torch(c.x), to_dev(c.ids), to_dev(c.weights)
    w13t, w2t = bits_to_torch(c.w13), bits_to_torch(c.w2)
    w13c, w13s = ctx.quantize_weight(w13t)
    w2c, w2s = ctx.quantize_weight(w2t)

    def run(rows):
        x_, i_, w_, d_ = (t[rows].contiguous() for t in (xt, ids, wts, dout))
        _, d = ctx.moe_fwd(x_, i_, w_, w13c, w13s, w2c, w2s, debug=True)
        return ctx.moe_bwd(x_, i_, w_, w13t, w2t, d["gate_up"], d["h"], d_)["dx"].clone()

    full = run(list(range(128)))
    for rows in ([0], [127], list(range(40, 72))):
        assert torch.equal(run(rows), full[rows])
