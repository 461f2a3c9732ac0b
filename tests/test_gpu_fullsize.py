"""GPU parity at the full benchmark sizes, in the launch configuration bench.py times, on
sampled outputs the oracle can compute one by one (teacher-forced on the GPU's own codes)."""
import os
import sys

import numpy as np
import pytest
import torch

import oracle
from paper_2604_07853_b200 import binding, build, inputs
from util import bf16_ulp_dist, bits_to_torch, torch_to_bits

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)
pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    build.build()
    c = binding.Context(0)
    yield c
    assert c.poll() == 0
    c.close()


def _tol(dec, ac, as_, wc, ws):
    ad = dec[ac] * np.repeat(as_.astype(np.float64), 128, axis=1)
    wd = dec[wc] * np.repeat(np.repeat(ws.astype(np.float64), 128, axis=0), 128, axis=1)
    return 1e-3 * np.linalg.norm(ad, axis=1)[:, None] * np.linalg.norm(wd, axis=1)[None, :]


def test_moe_training_shape_sampled(ctx):
    """M = 32768, Zipf(1.1): the exact tensors and call sequence of the benchmark step."""
    import bench
    dev = torch.device("cuda", 0)
    M, H, I, E, k = 32768, bench.H, bench.I, bench.E, bench.TOPK
    w13, w2, x, ids, wts = bench.make_inputs(M, 1000, dev, zipf=True)
    w13c, w13s = ctx.quantize_weight(w13)
    w2c, w2s = ctx.quantize_weight(w2)
    out, d = ctx.moe_fwd(x, ids, wts, w13c, w13s, w2c, w2s, debug=True)
    assert ctx.poll() == 0
    dec = oracle.e4m3_decode_table()
    ids_h, wts_h = ids.cpu().numpy(), wts.cpu().numpy()

    # weight quantization: three experts, bit-exact
    for e in (0, 57, 127):
        oc, os_ = oracle.quantize_weight(torch_to_bits(w13[e]))
        assert np.array_equal(w13c[e].cpu().numpy(), oc) and np.array_equal(w13s[e].cpu().numpy(), os_)
        oc, os_ = oracle.quantize_weight(torch_to_bits(w2[e]))
        assert np.array_equal(w2c[e].cpu().numpy(), oc) and np.array_equal(w2s[e].cpu().numpy(), os_)

    # permutation: bit-exact over all 262144 pairs
    off, srt, _ = oracle.permute(ids_h, E)
    assert np.array_equal(d["expert_offsets"].cpu().numpy(), off)
    assert np.array_equal(d["sorted_pair"].cpu().numpy(), srt)
    sizes = np.diff(off)
    assert sizes.sum() == M * k and sizes.max() > 10 * np.median(sizes)      # skewed, as intended

    # sampled sorted positions: the first and the last row of EVERY expert group (where a tile's mask
    # decides), the middle of the smallest, median and largest groups, and random ones: > 512 rows
    rng = np.random.default_rng(0)
    order = np.argsort(sizes)
    picks = []
    for e in range(E):
        if sizes[e] > 0:
            picks += [off[e], off[e + 1] - 1]
    for e in (order[np.nonzero(sizes[order])[0][0]], order[E // 2], order[-1]):
        picks.append((off[e] + off[e + 1]) // 2)
    picks += list(rng.integers(0, M * k, size=300))
    picks = np.array(sorted(set(int(q) for q in picks)))
    assert picks.size >= 512
    tok = srt[picks] // k
    exp = ids_h.reshape(-1)[srt[picks]]
    xs_bits = torch_to_bits(x[torch.from_numpy(tok).cuda()])
    xc, xs = oracle.quantize_act(xs_bits)
    gu = torch_to_bits(d["gate_up"][torch.from_numpy(picks).cuda()])
    hh = torch_to_bits(d["h"][torch.from_numpy(picks).cuda()])
    hc = d["h_codes"][torch.from_numpy(picks).cuda()].cpu().numpy()
    hs = d["h_scales"][torch.from_numpy(picks).cuda()].cpu().numpy()
    dn = d["down_f32"][torch.from_numpy(picks).cuda()].cpu().numpy()
    far = 0
    wcache = {}

    def weights_of(e):
        if e not in wcache:
            wcache.clear()                      # picks are sorted by position, hence by expert: keep one
            wcache[e] = (w13c[e].cpu().numpy(), w13s[e].cpu().numpy(), w2c[e].cpu().numpy(), w2s[e].cpu().numpy())
        return wcache[e]

    for i, e in enumerate(exp):
        a13, s13, a2, s2 = weights_of(int(e))
        o32, o16 = oracle.linear_q(xc[i:i + 1], xs[i:i + 1], a13, s13)
        dist = bf16_ulp_dist(gu[i:i + 1], o16)
        bad = dist > 1
        if bad.any():
            tol = _tol(dec, xc[i:i + 1], xs[i:i + 1], a13, s13)
            g = inputs.bf16_bits_to_f32(gu[i:i + 1]).astype(np.float64)
            assert (np.abs(g - o32)[bad] <= tol[bad] + np.abs(g[bad]) * 2.0 ** -8).all()
        far += int(bad.sum())
        assert bf16_ulp_dist(hh[i:i + 1], oracle.swiglu(gu[i:i + 1])).max() <= 1
        oc, os_ = oracle.quantize_act(hh[i:i + 1])
        assert np.array_equal(hc[i:i + 1], oc) and np.array_equal(hs[i:i + 1], os_)
        o32, _ = oracle.linear_q(hc[i:i + 1], hs[i:i + 1], a2, s2)
        tol = _tol(dec, hc[i:i + 1], hs[i:i + 1], a2, s2)
        assert (np.abs(dn[i:i + 1].astype(np.float64) - o32) <= tol).all()
    assert far <= 1e-3 * gu.size

    # combine: sampled tokens, bit-exact given the GPU's fp32 rows
    pos = np.empty(M * k, dtype=np.int64)
    pos[srt] = np.arange(M * k)
    for t in rng.integers(0, M, size=256):
        rows = torch.from_numpy(pos[t * k:(t + 1) * k]).cuda()
        y = d["down_f32"][rows].cpu().numpy()
        ref = oracle.combine(y, ids_h[t:t + 1], wts_h[t:t + 1])
        assert np.array_equal(torch_to_bits(out[t:t + 1]), ref)

    # sharding equivalence: the same tokens run as two halves give the same bytes
    half = M // 2
    a = ctx.moe_fwd(x[:half], ids[:half], wts[:half], w13c, w13s, w2c, w2s).clone()
    b = ctx.moe_fwd(x[half:], ids[half:], wts[half:], w13c, w13s, w2c, w2s)
    assert torch.equal(torch.cat([a, b]), out)


def test_qkv_projection_training_shape_sampled(ctx):
    """K = 2048, N = 5120, M = 8192: sampled rows against the oracle; M = 64 rows bitwise equal."""
    case = inputs.config2(8192)
    wc, ws = ctx.quantize_weight(bits_to_torch(case.w))
    oc, os_ = oracle.quantize_weight(case.w)
    assert np.array_equal(wc.cpu().numpy(), oc) and np.array_equal(ws.cpu().numpy(), os_)
    xt = bits_to_torch(case.x)
    y, y32 = ctx.linear_fwd(xt, wc, ws, want_f32=True)
    assert ctx.poll() == 0
    rows = np.array([0, 1, 127, 128, 129, 4095, 4096, 8190, 8191] + list(np.random.default_rng(1).integers(0, 8192, 23)))
    xc, xs = oracle.quantize_act(case.x[rows])
    o32, o16 = oracle.linear_q(xc, xs, oc, os_)
    dec = oracle.e4m3_decode_table()
    tol = _tol(dec, xc, xs, oc, os_)
    g32 = y32[torch.from_numpy(rows).cuda()].cpu().numpy()
    g16 = torch_to_bits(y[torch.from_numpy(rows).cuda()])
    err = np.abs(g32.astype(np.float64) - o32)
    assert (err <= tol).all()
    assert np.array_equal(g16, oracle.bf16_rne(g32))
    far = bf16_ulp_dist(g16, o16) > 1
    assert far.mean() < 1e-3 and (err[far] <= tol[far]).all()
    sub = ctx.linear_fwd(xt[:64].contiguous(), wc, ws)
    assert torch.equal(sub, y[:64])
