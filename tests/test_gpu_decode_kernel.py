"""The grouped FP8 GEMM has a wide-tile kernel and a swapped-operand kernel for decode-sized groups,
and a decode-sized layer runs both projections and the k-sum as one launch of the latter.
All must give the same bytes for every row (the fixed K-reduction order of App. C holds across
kernels, not only across batch sizes): one input goes through each, forced by the harness switch
(0 = automatic: the one-launch layer where it applies), and every stage the layer exposes is
compared bit for bit."""
import numpy as np
import pytest
import torch

from paper_2604_07853_b200 import binding, build, inputs
from util import bits_to_torch

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    build.build()
    c = binding.Context(0)
    yield c
    c.harness_set_gemm_path(0)
    c.close()


def _layer(ctx, c, path, debug=True):
    ctx.harness_set_gemm_path(path)
    w13c, w13s = ctx.quantize_weight(bits_to_torch(c.w13))
    w2c, w2s = ctx.quantize_weight(bits_to_torch(c.w2))
    r = ctx.moe_fwd(bits_to_torch(c.x), torch.from_numpy(c.ids).cuda(), torch.from_numpy(c.weights).cuda(),
                    w13c, w13s, w2c, w2s, debug=debug)
    assert ctx.poll() == 0
    ctx.harness_set_gemm_path(0)
    return r


@pytest.mark.parametrize("m,h,i,e,k", [(256, 2048, 768, 128, 8), (64, 512, 256, 8, 2), (1, 512, 256, 8, 2),
                                       (300, 384, 128, 4, 2), (8, 2048, 768, 128, 8), (33, 256, 384, 2, 1)])
def test_decode_kernel_equals_wide_kernel_stage_by_stage(ctx, m, h, i, e, k):
    c = inputs.moe_case(21, m, h=h, i=i, e=e, k=k)
    out_w, d_w = _layer(ctx, c, 1)
    P = m * k
    for path in (2, 0):
        out_d, d_d = _layer(ctx, c, path)
        for key in ("expert_offsets", "sorted_pair", "gate_up", "h", "h_codes", "h_scales", "down_f32"):
            a, b = d_w[key], d_d[key]
            assert torch.equal(a.view(torch.uint8), b.view(torch.uint8)), (path, key)
        assert torch.equal(out_w, out_d), path
    # and without the debug dumps
    wide = _layer(ctx, c, 1, debug=False)
    assert torch.equal(wide, _layer(ctx, c, 2, debug=False))
    assert torch.equal(wide, _layer(ctx, c, 0, debug=False))
    assert P > 0


def test_automatic_choice_matches_both(ctx):
    """Decode shape: the automatic path (the decode kernel at this size) against the forced wide one."""
    c = inputs.moe_case(3, 256)
    auto = _layer(ctx, c, 0, debug=False)
    wide = _layer(ctx, c, 1, debug=False)
    assert torch.equal(auto, wide)


def test_skewed_groups_through_the_decode_kernel(ctx):
    """Groups far larger than one 32-row chunk (and empty ones) through the decode kernel."""
    c = inputs.moe_case(5, 700, h=512, i=256, e=8, k=2, zipf_s=1.1)
    out_w, d_w = _layer(ctx, c, 1)
    out_d, d_d = _layer(ctx, c, 2)
    assert torch.equal(d_w["h_codes"], d_d["h_codes"]) and torch.equal(d_w["down_f32"].view(torch.int32), d_d["down_f32"].view(torch.int32))
    assert torch.equal(out_w, out_d)


@pytest.mark.parametrize("m,e,k,zipf", [(40, 64, 8, 0.0), (8, 128, 8, 0.0), (100, 16, 4, 1.1), (256, 128, 8, 1.1),
                                         (3, 128, 8, 0.0), (200, 40, 5, 1.5)])
def test_one_launch_layer_repeated_and_skewed(ctx, m, e, k, zipf):
    """The one-launch layer on shapes with many empty experts, experts of several 32-row chunks and
    fewer experts than the distance between an expert's two projections in its tile list; three
    calls in a row (its counters are cleared by the grouping kernel of each call)."""
    c = inputs.moe_case(77, m, h=512, i=256, e=e, k=k, zipf_s=zipf) if zipf else inputs.moe_case(77, m, h=512, i=256, e=e, k=k)
    ref, d_ref = _layer(ctx, c, 2)
    for _ in range(3):
        out, d = _layer(ctx, c, 0)
        assert torch.equal(d_ref["h_codes"], d["h_codes"]) and torch.equal(d_ref["h_scales"], d["h_scales"])
        assert torch.equal(d_ref["down_f32"].view(torch.int32), d["down_f32"].view(torch.int32))
        assert torch.equal(ref, out)
        assert torch.equal(ref, _layer(ctx, c, 0, debug=False))


@pytest.mark.parametrize("m,h,i,e,k", [(24, 4096, 1536, 16, 4), (40, 1024, 128, 300, 6), (17, 8192, 256, 4, 2)])
def test_one_launch_layer_long_k_and_many_experts(ctx, m, h, i, e, k):
    """K up to the scale slab's limit (64 K-blocks), an expert count that is no power of two and exceeds
    one byte, a down projection of a single K-block."""
    c = inputs.moe_case(91, m, h=h, i=i, e=e, k=k)
    wide, d_w = _layer(ctx, c, 1)
    out, d = _layer(ctx, c, 0)
    for key in ("expert_offsets", "sorted_pair", "gate_up", "h", "h_codes", "h_scales", "down_f32"):
        assert torch.equal(d_w[key].view(torch.uint8), d[key].view(torch.uint8)), key
    assert torch.equal(wide, out)


def test_decode_step_replays_from_a_cuda_graph(ctx):
    """The decode-sized layer call allocates nothing and synchronizes nothing, so a stream capture
    takes it whole (its launches keep their programmatic dependencies); replaying the graph gives the
    bytes of the plain call, also after the output and the workspace were overwritten in between."""
    c = inputs.moe_case(13, 256)
    w13c, w13s = ctx.quantize_weight(bits_to_torch(c.w13))
    w2c, w2s = ctx.quantize_weight(bits_to_torch(c.w2))
    x, ids, wts = bits_to_torch(c.x), torch.from_numpy(c.ids).cuda(), torch.from_numpy(c.weights).cuda()
    M, H = x.shape
    out = torch.empty((M, H), dtype=torch.bfloat16, device=x.device)
    ws = torch.empty(ctx.moe_workspace_bytes(M, H, w2c.shape[2], w13c.shape[0], ids.shape[1]), dtype=torch.uint8,
                     device=x.device)
    ref = ctx.moe_fwd(x, ids, wts, w13c, w13s, w2c, w2s).clone()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        ctx.moe_fwd(x, ids, wts, w13c, w13s, w2c, w2s, out=out, workspace=ws)
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g, stream=side):
        for _ in range(3):
            ctx.moe_fwd(x, ids, wts, w13c, w13s, w2c, w2s, out=out, workspace=ws)
    for _ in range(2):
        out.zero_()
        ws.fill_(0xA5)
        g.replay()
        torch.cuda.synchronize()
        assert torch.equal(out, ref) and ctx.poll() == 0


@pytest.mark.parametrize("m,n,k", [(64, 5120, 2048), (1, 256, 512), (31, 384, 128), (33, 128, 1024), (64, 2048, 4096),
                                   (17, 640, 3968)])
def test_dense_projection_decode_kernel_equals_wide_kernel(ctx, m, n, k):
    """A dense projection of at most 64 rows runs on the swapped-operand kernel (automatic choice and
    forced), larger ones on the wide-tile kernel: bf16 rows and fp32 accumulators must be the same bytes,
    and a row's bytes must not depend on the batch around it."""
    c = inputs.linear_case(300 + m, m, n, k)
    wc, ws = ctx.quantize_weight(bits_to_torch(c.w))
    x = bits_to_torch(c.x)
    y0, f0 = ctx.linear_fwd(x, wc, ws, want_f32=True)
    plain = ctx.linear_fwd(x, wc, ws).clone()
    assert ctx.poll() == 0
    for path in (1, 2):
        ctx.harness_set_gemm_path(path)
        y, f = ctx.linear_fwd(x, wc, ws, want_f32=True)
        ctx.harness_set_gemm_path(0)
        assert ctx.poll() == 0
        assert torch.equal(y0, y) and torch.equal(f0.view(torch.int32), f.view(torch.int32)), path
    assert torch.equal(plain, y0)
    for rows in ([0], [m - 1], list(range(m // 2, m))):
        assert torch.equal(ctx.linear_fwd(x[rows].contiguous(), wc, ws), y0[rows])
