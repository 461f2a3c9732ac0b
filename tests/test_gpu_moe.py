"""GPU parity: qarl_moe_fwd against the oracle (stage by stage, teacher-forced) and the
bitwise row invariance of the layer across batch compositions."""
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


class DeviceCase:
    def __init__(self, ctx, case):
        self.case = case
        self.x = bits_to_torch(case.x)
        self.ids = to_dev(case.ids)
        self.wts = to_dev(case.weights)
        self.w13c, self.w13s = ctx.quantize_weight(bits_to_torch(case.w13))
        self.w2c, self.w2s = ctx.quantize_weight(bits_to_torch(case.w2))

    def run(self, ctx, debug=False, rows=None):
        x, ids, wts = self.x, self.ids, self.wts
        if rows is not None:
            x, ids, wts = x[rows].contiguous(), ids[rows].contiguous(), wts[rows].contiguous()
        return ctx.moe_fwd(x, ids, wts, self.w13c, self.w13s, self.w2c, self.w2s, debug=debug)


def _tol(dec, ac, as_, wc, ws):
    ad = dec[ac] * np.repeat(as_.astype(np.float64), 128, axis=1)
    wd = dec[wc] * np.repeat(np.repeat(ws.astype(np.float64), 128, axis=0), 128, axis=1)
    return 1e-3 * np.linalg.norm(ad, axis=1)[:, None] * np.linalg.norm(wd, axis=1)[None, :]


def check_moe(ctx, case, end_to_end=True):
    dc = DeviceCase(ctx, case)
    out, d = dc.run(ctx, debug=True)
    assert ctx.poll() == 0
    c = case
    P = c.M * c.k
    dec = oracle.e4m3_decode_table()
    w13c, w13s, w2c, w2s = (t.cpu().numpy() for t in (dc.w13c, dc.w13s, dc.w2c, dc.w2s))

    # 1. permutation: bit-exact
    off, srt, _ = oracle.permute(c.ids, c.E)
    assert np.array_equal(d["expert_offsets"].cpu().numpy(), off)
    assert np.array_equal(d["sorted_pair"].cpu().numpy(), srt)

    # 2. gate_up (sorted order) vs the oracle on the GPU's own activation codes
    xc, xs = ctx.quantize_act(dc.x)
    xc, xs = xc.cpu().numpy(), xs.cpu().numpy()
    oc, os_ = oracle.quantize_act(c.x)
    assert np.array_equal(xc, oc) and np.array_equal(xs, os_)
    tok = srt // c.k
    gu_gpu = torch_to_bits(d["gate_up"])
    stats = dict(gu_far=0, gu_n=0)
    for e in range(c.E):
        a, b = off[e], off[e + 1]
        if a == b:
            continue
        o32, o16 = oracle.linear_q(xc[tok[a:b]], xs[tok[a:b]], w13c[e], w13s[e])
        dist = bf16_ulp_dist(gu_gpu[a:b], o16)
        far = dist > 1
        if far.any():
            tol = _tol(dec, xc[tok[a:b]], xs[tok[a:b]], w13c[e], w13s[e])
            g = inputs.bf16_bits_to_f32(gu_gpu[a:b]).astype(np.float64)
            # a bf16 value sits within half an ulp of the fp32 it was rounded from
            ulp = np.abs(g) * 2.0 ** -8
            assert (np.abs(g - o32)[far] <= tol[far] + ulp[far]).all()
        stats["gu_far"] += int(far.sum())
        stats["gu_n"] += far.size
    assert stats["gu_far"] <= 1e-3 * stats["gu_n"]

    # 3. SwiGLU: oracle applied to the GPU's gate_up, <= 1 bf16 ulp
    h_gpu = torch_to_bits(d["h"])
    h_or = oracle.swiglu(gu_gpu)
    assert bf16_ulp_dist(h_gpu, h_or).max() <= 1
    assert (h_gpu == h_or).mean() > 0.99

    # 4. fused re-quantization: bit-exact on the GPU's own h
    hc, hs = oracle.quantize_act(h_gpu)
    assert np.array_equal(d["h_codes"].cpu().numpy(), hc)
    assert np.array_equal(d["h_scales"].cpu().numpy().view(np.uint32), hs.view(np.uint32))

    # 5. down projection (fp32, sorted order) vs the oracle on the GPU's h codes
    dn = d["down_f32"].cpu().numpy()
    for e in range(c.E):
        a, b = off[e], off[e + 1]
        if a == b:
            continue
        o32, _ = oracle.linear_q(hc[a:b], hs[a:b], w2c[e], w2s[e])
        tol = _tol(dec, hc[a:b], hs[a:b], w2c[e], w2s[e])
        err = np.abs(dn[a:b].astype(np.float64) - o32)
        assert (err <= tol).all(), f"expert {e}: max err/tol {(err / tol).max()}"

    # 6. combine: exact arithmetic on the GPU's fp32 rows -> bit-exact
    by_pair = np.empty_like(dn)
    by_pair[srt] = dn
    assert np.array_equal(torch_to_bits(out), oracle.combine(by_pair, c.ids, c.weights))

    # 7. end to end against the independent oracle (informational bounds)
    if end_to_end:
        ref = oracle.moe(c.x, c.ids, c.weights, w13c, w13s, w2c, w2s)
        g = inputs.bf16_bits_to_f32(torch_to_bits(out)).astype(np.float64)
        r = inputs.bf16_bits_to_f32(ref).astype(np.float64)
        rel = np.linalg.norm(g - r) / np.linalg.norm(r)
        dist = bf16_ulp_dist(torch_to_bits(out), ref)
        stats.update(rel=float(rel), exact=float((dist == 0).mean()), within1=float((dist <= 1).mean()))
        assert rel < 5e-3, stats
    return stats


def test_small_layer(ctx):
    check_moe(ctx, inputs.moe_case(5, 24, h=256, i=128, e=8, k=2))


def test_ragged_groups_and_empty_experts(ctx):
    # 3 tokens over 16 experts: most experts empty; 333 tokens: groups straddle 128-row tiles
    check_moe(ctx, inputs.moe_case(6, 3, h=256, i=256, e=16, k=4))
    check_moe(ctx, inputs.moe_case(7, 333, h=512, i=256, e=4, k=2))


def test_skewed_popularity_multi_chunk(ctx):
    # P = 1200 * 8 = 9600 pairs: several permutation chunks, Zipf-skewed group sizes
    check_moe(ctx, inputs.moe_case(8, 1200, h=256, i=128, e=32, k=8, zipf_s=1.1), end_to_end=False)


def test_config3_decode_layer(ctx):
    stats = check_moe(ctx, inputs.config3())
    assert stats["within1"] > 0.98


def test_row_invariance_across_batch_compositions(ctx):
    """App. C: every token's output row is bitwise identical whatever the batch it runs in."""
    case = inputs.moe_case(9, 200, h=512, i=256, e=16, k=4)
    dc = DeviceCase(ctx, case)
    full = dc.run(ctx).clone()
    rng = np.random.default_rng(0)
    for m in (1, 2, 8, 64, 130):
        perm = rng.permutation(case.M)
        for start in range(0, min(case.M, 3 * m), m):
            rows = torch.from_numpy(perm[start:start + m].copy()).cuda()
            sub = dc.run(ctx, rows=rows)
            assert torch.equal(sub, full[rows]), (m, start)
    assert ctx.poll() == 0


def test_slot_order_does_not_matter(ctx):
    case = inputs.moe_case(10, 40, h=256, i=128, e=8, k=4)
    dc = DeviceCase(ctx, case)
    base = dc.run(ctx).clone()
    perm = torch.tensor([2, 0, 3, 1], device="cuda")
    dc.ids = dc.ids[:, perm].contiguous()
    dc.wts = dc.wts[:, perm].contiguous()
    assert torch.equal(dc.run(ctx), base)


def test_k1_reduces_to_two_linear_calls(ctx):
    """k = 1, weight 1: the layer is gate_up linear -> SwiGLU -> down linear; the fused path's
    dumps must equal the library's own dense entry points bit for bit."""
    case = inputs.moe_case(11, 50, h=256, i=128, e=4, k=1)
    case.weights[:] = 1.0
    dc = DeviceCase(ctx, case)
    out, d = dc.run(ctx, debug=True)
    srt = d["sorted_pair"].cpu().numpy()
    off = d["expert_offsets"].cpu().numpy()
    for e in range(case.E):
        a, b = off[e], off[e + 1]
        if a == b:
            continue
        rows = torch.from_numpy(srt[a:b].copy()).cuda()
        gu = ctx.linear_fwd(dc.x[rows].contiguous(), dc.w13c[e], dc.w13s[e])
        assert torch.equal(gu, d["gate_up"][a:b])
        y = ctx.linear_fwd_q(d["h_codes"][a:b].contiguous(), d["h_scales"][a:b].contiguous(),
                             dc.w2c[e], dc.w2s[e])
        assert torch.equal(y, out[rows])


def test_bad_expert_ids_are_reported_not_fatal(ctx):
    case = inputs.moe_case(12, 16, h=256, i=128, e=8, k=2)
    dc = DeviceCase(ctx, case)
    good = dc.run(ctx).clone()
    ids = dc.ids.clone()
    dc.ids = ids.clone()
    dc.ids[3, 1] = 99
    dc.run(ctx)
    assert ctx.poll() == -8
    dc.ids = ids.clone()
    dc.ids[5, 1] = dc.ids[5, 0]
    dc.run(ctx)
    assert ctx.poll() == -8
    dc.ids = ids
    assert torch.equal(dc.run(ctx), good) and ctx.poll() == 0


def test_empty_batch_and_argument_errors(ctx):
    case = inputs.moe_case(13, 4, h=256, i=128, e=4, k=2)
    dc = DeviceCase(ctx, case)
    out = ctx.moe_fwd(dc.x[:0], dc.ids[:0], dc.wts[:0], dc.w13c, dc.w13s, dc.w2c, dc.w2s)
    assert out.shape == (0, 256)
    small = torch.empty(256, dtype=torch.uint8, device="cuda")
    with pytest.raises(binding.QarlError) as ei:
        ctx.moe_fwd(dc.x, dc.ids, dc.wts, dc.w13c, dc.w13s, dc.w2c, dc.w2s, workspace=small)
    assert ei.value.status == -4


def test_layer_can_be_captured_in_a_cuda_graph(ctx):
    """The layer makes no allocation, no synchronisation and no host read between its launches, so a
    stream capture records it; a replay gives the bytes of the eager call."""
    c = inputs.moe_case(13, 64, h=256, i=128, e=8, k=2)
    dc = DeviceCase(ctx, c)
    ref = dc.run(ctx).clone()
    out = torch.empty_like(ref)
    ws = ctx.workspace(ctx.moe_workspace_bytes(c.M, c.H, c.I, c.E, c.k))
    s = torch.cuda.Stream()
    with torch.cuda.stream(s):
        ctx.moe_fwd(dc.x, dc.ids, dc.wts, dc.w13c, dc.w13s, dc.w2c, dc.w2s, out=out, workspace=ws)
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g, stream=s):
        ctx.moe_fwd(dc.x, dc.ids, dc.wts, dc.w13c, dc.w13s, dc.w2c, dc.w2s, out=out, workspace=ws)
    out.zero_()
    g.replay()
    torch.cuda.synchronize()
    assert torch.equal(out, ref)
    assert ctx.poll() == 0
