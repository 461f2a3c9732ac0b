"""GPU parity of the W4A16 path (Sec. 2.2, integer quantization; weight-only 4-bit with bf16
activations): quantizer bit-exact against the oracle, the GEMM and the MoE layer teacher-forced
against the oracle on the GPU's own codes, and the bitwise row invariance across batch shapes."""
import numpy as np
import pytest
import torch

import oracle
from paper_2604_07853_b200 import binding, build, inputs
from util import bf16_ulp_dist, bits_to_torch, to_dev, torch_to_bits

pytestmark = pytest.mark.gpu

# element held by nibble p of a 32-bit word in the library's storage order
_NIBBLE_ELEM = np.array([0, 2, 4, 6, 1, 3, 5, 7])


@pytest.fixture(scope="module")
def ctx():
    build.build()
    c = binding.Context(0)
    yield c
    assert c.poll() == 0
    c.close()


def unpack_lib(packed: np.ndarray) -> np.ndarray:
    """library storage [.., N, K/2] u8 (tile-major 4 KB chunks) -> codes [.., N, K]: pure re-ordering."""
    *lead, N, K2 = packed.shape
    K = K2 * 2
    words = np.ascontiguousarray(packed).reshape(-1).view("<u4")
    # [.., N/128 blocks, K/64 steps, quad 2, row 128, word-in-quad 4]
    words = words.reshape(-1, N // 128, K // 64, 2, 128, 4)
    words = words.transpose(0, 1, 4, 2, 3, 5).reshape(-1, N, K // 8)      # [.., row, word along K]
    nib = np.stack([(words >> (4 * p)) & 15 for p in range(8)], axis=-1).astype(np.uint8)
    codes = np.empty_like(nib)
    codes[..., _NIBBLE_ELEM] = nib
    return codes.reshape(*lead, N, K)


def unpack_linear(packed: np.ndarray) -> np.ndarray:
    """oracle storage (code 2j low nibble, 2j+1 high nibble of byte j) -> codes [.., K]."""
    return np.stack([packed & 15, packed >> 4], axis=-1).reshape(*packed.shape[:-1], packed.shape[-1] * 2)


def pack_linear(codes: np.ndarray) -> np.ndarray:
    c = codes.reshape(*codes.shape[:-1], codes.shape[-1] // 2, 2)
    return (c[..., 0] | (c[..., 1] << 4)).astype(np.uint8)


def host_weights(q):
    """GPU (packed, scales, zeros) -> oracle-layout (packed, scales f32 [.., N, K/128], zeros)."""
    packed, scales, zeros = q
    p = pack_linear(unpack_lib(packed.cpu().numpy()))
    s = inputs.bf16_bits_to_f32(torch_to_bits(scales))
    return p, np.ascontiguousarray(np.swapaxes(s, -1, -2)), np.ascontiguousarray(np.swapaxes(zeros.cpu().numpy(), -1, -2))


def w_hat_of(q):
    return oracle.dequant_w4(*host_weights(q))


class Int4:
    """The calls of the integer format, so that the checks below also serve the e2m1 format."""
    @staticmethod
    def quantize(ctx, w):
        return ctx.quantize_weight_w4(w)

    @staticmethod
    def linear(ctx, x, q, **kw):
        return ctx.linear_fwd_w4a16(x, *q, **kw)

    @staticmethod
    def moe(ctx, x, ids, wts, q13, q2, **kw):
        return ctx.moe_fwd_w4a16(x, ids, wts, q13, q2, **kw)

    w_hat = staticmethod(w_hat_of)


# ------------------------------------------------------------------------------ quantizer
@pytest.mark.parametrize("e,n,k", [(1, 128, 128), (3, 256, 384), (2, 1536, 2048), (4, 640, 256)])
def test_quantizer_bit_exact(ctx, e, n, k):
    rng = np.random.default_rng(10 + n)
    w = inputs.weight_bf16(rng, e, n, k)
    w[0, 0, :128] = 0                      # an all-zero group
    w[-1, -1, ::3] = 0
    op, os_, oz = oracle.quantize_weight_w4(w)
    gp, gs, gz = host_weights(ctx.quantize_weight_w4(bits_to_torch(w)))
    assert np.array_equal(unpack_linear(gp), unpack_linear(op))
    assert np.array_equal(gs.view(np.uint32), os_.view(np.uint32))
    assert np.array_equal(gz, oz)


def test_quantizer_all_positive_and_all_negative_groups(ctx):
    rng = np.random.default_rng(3)
    w = inputs.bf16_bits_to_f32(inputs.weight_bf16(rng, 1, 128, 256))
    w[:, :64, :128] = np.abs(w[:, :64, :128]) + 0.01     # lo clamps to 0: z = 0
    w[:, 64:, 128:] = -np.abs(w[:, 64:, 128:]) - 0.01    # hi clamps to 0: z = 15
    wb = inputs.f32_to_bf16_bits(w)
    op, os_, oz = oracle.quantize_weight_w4(wb)
    gp, gs, gz = host_weights(ctx.quantize_weight_w4(bits_to_torch(wb)))
    assert (oz[0, :64, 0] == 0).all() and (oz[0, 64:, 1] == 15).all()
    assert np.array_equal(unpack_linear(gp), unpack_linear(op))
    assert np.array_equal(gs, os_) and np.array_equal(gz, oz)


def test_quantizer_exact_ties_round_to_even(ctx):
    """Multiples of s/2: every other value sits exactly half-way between two codes, where the
    result must be the even neighbour (the oracle's rint of an exact IEEE quotient)."""
    rng = np.random.default_rng(5)
    w = rng.integers(-16, 15, size=(1, 128, 384)).astype(np.float32) * 0.125     # s = 3.75 / 15 = 0.25
    w[:, :, ::128] = -2.0
    w[:, :, 1::128] = 1.75
    # other scales: the same pattern times powers of two and times 3 (s keeps 8 significant bits)
    w[:, 32:64] *= 8.0
    w[:, 64:96] *= 2.0 ** -10
    w[:, 96:] *= 3.0
    wb = inputs.f32_to_bf16_bits(w)
    assert np.array_equal(inputs.bf16_bits_to_f32(wb), w)
    op, os_, oz = oracle.quantize_weight_w4(wb)
    assert os_[0, 0, 0] == np.float32(0.25) and os_[0, 100, 0] == np.float32(0.75)
    gp, gs, gz = host_weights(ctx.quantize_weight_w4(bits_to_torch(wb)))
    assert np.array_equal(unpack_linear(gp), unpack_linear(op))
    assert np.array_equal(gs, os_) and np.array_equal(gz, oz)


def test_quantizer_publish_writes_two_equal_copies(ctx):
    """Sec. 3.1 item 3: the published 4-bit tensors are the ones the training forward uses, bit for bit."""
    rng = np.random.default_rng(8)
    wt = bits_to_torch(inputs.weight_bf16(rng, 2, 256, 384))
    ref = ctx.quantize_weight_w4(wt)
    a = tuple(torch.zeros_like(t) for t in ref)
    b = tuple(torch.zeros_like(t) for t in ref)
    ctx.quantize_weight_w4_publish(wt, a, b)
    for r, x, y in zip(ref, a, b):
        assert torch.equal(r, x) and torch.equal(r, y)


# ------------------------------------------------------------------------------ dense GEMM
def check_linear(ctx, seed, m, n, k, fmt=Int4):
    """fp32: |gpu - oracle| <= 1e-3 * ||x_row|| * ||w^_col|| (the oracle sums exactly; the tensor
    core adds K exact products in fp32).  bf16: the rounding of the GPU's own fp32, bit for bit,
    and within 1 ulp of the oracle's except where cancellation makes an ulp smaller than the
    fp32 bound (rare)."""
    case = inputs.linear_case(seed, m, n, k)
    q = fmt.quantize(ctx, bits_to_torch(case.w))
    xt = bits_to_torch(case.x)
    y, y32 = fmt.linear(ctx, xt, q, want_f32=True)
    assert ctx.poll() == 0
    w_hat = fmt.w_hat(q)
    o32, o16 = oracle.linear_bf16(case.x, w_hat)
    g32, g16 = y32.cpu().numpy(), torch_to_bits(y)
    nx = np.linalg.norm(inputs.bf16_bits_to_f32(case.x).astype(np.float64), axis=1)
    nw = np.linalg.norm(inputs.bf16_bits_to_f32(w_hat).astype(np.float64), axis=1)
    tol = 1e-3 * nx[:, None] * nw[None, :]
    err = np.abs(g32.astype(np.float64) - o32.astype(np.float64))
    assert (err <= tol).all(), f"max err/tol = {(err / tol).max()}"
    assert np.array_equal(g16, oracle.bf16_rne(g32))
    far = bf16_ulp_dist(g16, o16) > 1
    assert far.mean() < 1e-3, f"{far.sum()} elements beyond 1 ulp"
    return float((err / tol).max())


@pytest.mark.parametrize("m,n,k", [(1, 128, 128), (127, 256, 256), (128, 384, 512), (129, 640, 2048),
                                   (300, 1280, 768), (5, 256, 4096), (70, 4096, 2048)])
def test_linear_shapes_and_ragged_tails(ctx, m, n, k):
    check_linear(ctx, 200 + m, m, n, k)


def test_linear_exact_on_integer_data(ctx):
    """Small integers: every product and partial sum is exact in fp32, so the GPU must match the
    exact result bit for bit (a wrong nibble, scale, zero point or swizzle cannot hide)."""
    rng = np.random.default_rng(4)
    m, n, k = 37, 256, 384
    x = inputs.f32_to_bf16_bits(rng.integers(-4, 5, size=(m, k)).astype(np.float32))
    # rows spanning exactly -8..7 quantize to s = 1, z = 8 and reproduce the integers exactly
    wf = rng.integers(-8, 8, size=(n, k)).astype(np.float32)
    wf[:, ::128] = -8
    wf[:, 1::128] = 7
    w = inputs.f32_to_bf16_bits(wf)
    q = ctx.quantize_weight_w4(bits_to_torch(w))
    assert np.array_equal(inputs.bf16_bits_to_f32(w_hat_of(q)), wf)
    _, y32 = ctx.linear_fwd_w4a16(bits_to_torch(x), *q, want_f32=True)
    assert np.array_equal(y32.cpu().numpy(), inputs.bf16_bits_to_f32(x) @ wf.T)


def test_linear_rows_do_not_depend_on_the_batch(ctx):
    case = inputs.linear_case(9, 300, 512, 1024)
    q = ctx.quantize_weight_w4(bits_to_torch(case.w))
    xt = bits_to_torch(case.x)
    full = ctx.linear_fwd_w4a16(xt, *q)
    for rows in ([0], [299], list(range(120, 140)), list(range(0, 300, 7))):
        part = ctx.linear_fwd_w4a16(xt[rows].contiguous(), *q)
        assert torch.equal(part, full[rows])


# ------------------------------------------------------------------------------ MoE layer
class DeviceCase:
    def __init__(self, ctx, case, fmt=Int4):
        self.case = case
        self.fmt = fmt
        self.x = bits_to_torch(case.x)
        self.ids = to_dev(case.ids)
        self.wts = to_dev(case.weights)
        self.w13 = fmt.quantize(ctx, bits_to_torch(case.w13))
        self.w2 = fmt.quantize(ctx, bits_to_torch(case.w2))

    def run(self, ctx, debug=False, rows=None):
        x, ids, wts = self.x, self.ids, self.wts
        if rows is not None:
            x, ids, wts = x[rows].contiguous(), ids[rows].contiguous(), wts[rows].contiguous()
        return self.fmt.moe(ctx, x, ids, wts, self.w13, self.w2, debug=debug)


def _norm_tol(a_bits, w_hat_bits):
    na = np.linalg.norm(inputs.bf16_bits_to_f32(a_bits).astype(np.float64), axis=1)
    nw = np.linalg.norm(inputs.bf16_bits_to_f32(w_hat_bits).astype(np.float64), axis=1)
    return 1e-3 * na[:, None] * nw[None, :]


def check_moe(ctx, case, end_to_end=True, fmt=Int4):
    dc = DeviceCase(ctx, case, fmt)
    out, d = dc.run(ctx, debug=True)
    assert ctx.poll() == 0
    c = case
    w13h, w2h = fmt.w_hat(dc.w13), fmt.w_hat(dc.w2)

    # 1. permutation: bit-exact
    off, srt, _ = oracle.permute(c.ids, c.E)
    assert np.array_equal(d["expert_offsets"].cpu().numpy(), off)
    assert np.array_equal(d["sorted_pair"].cpu().numpy(), srt)

    # 2. gate_up (sorted order): <= 1 bf16 ulp of the oracle, beyond that only inside the fp32 bound
    tok = srt // c.k
    gu_gpu = torch_to_bits(d["gate_up"])
    n_far = 0
    for e in range(c.E):
        a, b = off[e], off[e + 1]
        if a == b:
            continue
        o32, o16 = oracle.linear_bf16(c.x[tok[a:b]], w13h[e])
        far = bf16_ulp_dist(gu_gpu[a:b], o16) > 1
        if far.any():
            tol = _norm_tol(c.x[tok[a:b]], w13h[e])
            g = inputs.bf16_bits_to_f32(gu_gpu[a:b]).astype(np.float64)
            assert (np.abs(g - o32)[far] <= tol[far] + np.abs(g[far]) * 2.0 ** -8).all()
        n_far += int(far.sum())
    assert n_far <= 1e-3 * gu_gpu.size

    # 3. SwiGLU on the GPU's own gate_up: <= 1 bf16 ulp
    h_gpu = torch_to_bits(d["h"])
    h_or = oracle.swiglu(gu_gpu)
    assert bf16_ulp_dist(h_gpu, h_or).max() <= 1
    assert (h_gpu == h_or).mean() > 0.99

    # 4. down projection (fp32, sorted order) on the GPU's own h
    dn = d["down_f32"].cpu().numpy()
    for e in range(c.E):
        a, b = off[e], off[e + 1]
        if a == b:
            continue
        o32, _ = oracle.linear_bf16(h_gpu[a:b], w2h[e])
        tol = _norm_tol(h_gpu[a:b], w2h[e])
        err = np.abs(dn[a:b].astype(np.float64) - o32)
        assert (err <= tol).all(), f"expert {e}: max err/tol {(err / tol).max()}"

    # 5. combine: exact arithmetic on the GPU's fp32 rows -> bit-exact
    by_pair = np.empty_like(dn)
    by_pair[srt] = dn
    assert np.array_equal(torch_to_bits(out), oracle.combine(by_pair, c.ids, c.weights))

    # 6. end to end against the independent oracle
    stats = {}
    if end_to_end:
        ref = oracle.moe_w4a16(c.x, c.ids, c.weights, w13h, w2h)
        g = inputs.bf16_bits_to_f32(torch_to_bits(out)).astype(np.float64)
        r = inputs.bf16_bits_to_f32(ref).astype(np.float64)
        rel = np.linalg.norm(g - r) / np.linalg.norm(r)
        dist = bf16_ulp_dist(torch_to_bits(out), ref)
        stats.update(rel=float(rel), exact=float((dist == 0).mean()), within1=float((dist <= 1).mean()))
        assert rel < 5e-3, stats
    return stats


def test_moe_small_layer(ctx):
    check_moe(ctx, inputs.moe_case(5, 24, h=256, i=128, e=8, k=2))


def test_moe_ragged_groups_and_empty_experts(ctx):
    check_moe(ctx, inputs.moe_case(6, 3, h=256, i=256, e=16, k=4))
    check_moe(ctx, inputs.moe_case(7, 333, h=512, i=256, e=4, k=2))


def test_moe_skewed_popularity(ctx):
    check_moe(ctx, inputs.moe_case(8, 1200, h=256, i=128, e=32, k=8, zipf_s=1.1), end_to_end=False)


def test_moe_decode_layer_shape(ctx):
    stats = check_moe(ctx, inputs.config3())
    assert stats["within1"] > 0.98


def test_moe_rows_do_not_depend_on_the_batch(ctx):
    case = inputs.moe_case(11, 256, h=512, i=256, e=16, k=4, zipf_s=1.1)
    dc = DeviceCase(ctx, case)
    full = dc.run(ctx)
    for rows in ([0], [255], list(range(100, 164)), list(range(0, 256, 5))):
        assert torch.equal(dc.run(ctx, rows=rows), full[rows])


# ------------------------------------------------------------------------------ full size
def test_moe_training_shape_sampled(ctx):
    """M = 32768, Zipf(1.1), the shapes of the benchmark step: sampled sorted positions against
    the oracle (teacher-forced on the GPU's own codes and intermediates), combine bit-exact on
    sampled tokens, and the same tokens run as two halves give the same bytes."""
    import os
    import sys
    sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
    import bench
    dev = torch.device("cuda", 0)
    M, H, I, E, k = 32768, bench.H, bench.I, bench.E, bench.TOPK
    w13, w2, x, ids, wts = bench.make_inputs(M, 1000, dev, zipf=True)
    q13 = ctx.quantize_weight_w4(w13)
    q2 = ctx.quantize_weight_w4(w2)
    out, d = ctx.moe_fwd_w4a16(x, ids, wts, q13, q2, debug=True)
    assert ctx.poll() == 0
    ids_h, wts_h = ids.cpu().numpy(), wts.cpu().numpy()

    # weight quantization: three experts, bit-exact (codes, scales, zero points)
    p13, s13, z13 = host_weights(q13)
    p2, s2, z2 = host_weights(q2)
    for e in (0, 57, 127):
        for w, (gp, gs, gz) in ((w13, (p13, s13, z13)), (w2, (p2, s2, z2))):
            op, os_, oz = oracle.quantize_weight_w4(torch_to_bits(w[e]))
            assert np.array_equal(gp[e], op) and np.array_equal(gs[e], os_) and np.array_equal(gz[e], oz)

    off, srt, _ = oracle.permute(ids_h, E)
    assert np.array_equal(d["expert_offsets"].cpu().numpy(), off)
    assert np.array_equal(d["sorted_pair"].cpu().numpy(), srt)
    sizes = np.diff(off)

    rng = np.random.default_rng(0)
    order = np.argsort(sizes)
    picks = []
    for e in (order[np.nonzero(sizes[order])[0][0]], order[E // 2], order[-1]):
        picks += [off[e], off[e + 1] - 1, (off[e] + off[e + 1]) // 2, off[e] + min(129, sizes[e] - 1)]
    picks += list(rng.integers(0, M * k, size=40))
    picks = np.array(sorted(set(int(q) for q in picks)))
    tok = srt[picks] // k
    exp = ids_h.reshape(-1)[srt[picks]]
    sel = torch.from_numpy(picks).cuda()
    xs_bits = torch_to_bits(x[torch.from_numpy(tok).cuda()])
    gu = torch_to_bits(d["gate_up"][sel])
    hh = torch_to_bits(d["h"][sel])
    dn = d["down_f32"][sel].cpu().numpy()
    far = 0
    what = {}
    for i, e in enumerate(exp):
        if e not in what:
            what[e] = (oracle.dequant_w4(p13[e], s13[e], z13[e]), oracle.dequant_w4(p2[e], s2[e], z2[e]))
        w13h, w2h = what[e]
        o32, o16 = oracle.linear_bf16(xs_bits[i:i + 1], w13h)
        bad = bf16_ulp_dist(gu[i:i + 1], o16) > 1
        if bad.any():
            tol = _norm_tol(xs_bits[i:i + 1], w13h)
            g = inputs.bf16_bits_to_f32(gu[i:i + 1]).astype(np.float64)
            assert (np.abs(g - o32)[bad] <= tol[bad] + np.abs(g[bad]) * 2.0 ** -8).all()
        far += int(bad.sum())
        assert bf16_ulp_dist(hh[i:i + 1], oracle.swiglu(gu[i:i + 1])).max() <= 1
        o32, _ = oracle.linear_bf16(hh[i:i + 1], w2h)
        assert (np.abs(dn[i:i + 1].astype(np.float64) - o32) <= _norm_tol(hh[i:i + 1], w2h)).all()
    assert far <= 1e-3 * gu.size

    pos = np.empty(M * k, dtype=np.int64)
    pos[srt] = np.arange(M * k)
    for t in rng.integers(0, M, size=24):
        rows = torch.from_numpy(pos[t * k:(t + 1) * k]).cuda()
        ref = oracle.combine(d["down_f32"][rows].cpu().numpy(), ids_h[t:t + 1], wts_h[t:t + 1])
        assert np.array_equal(torch_to_bits(out[t:t + 1]), ref)

    half = M // 2
    a = ctx.moe_fwd_w4a16(x[:half], ids[:half], wts[:half], q13, q2).clone()
    b = ctx.moe_fwd_w4a16(x[half:], ids[half:], wts[half:], q13, q2)
    assert torch.equal(torch.cat([a, b]), out)
    # decode-sized call on a slice of the same tokens (128-row tiles) gives the same rows
    c = ctx.moe_fwd_w4a16(x[:256], ids[:256], wts[:256], q13, q2)
    assert torch.equal(c, out[:256])
