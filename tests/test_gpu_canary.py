"""Memory-safety checks that stand in for a sanitizer: every buffer a call may write (outputs and
workspace) sits inside a larger buffer filled with a poison byte, and the poison around it must be
intact afterwards.  Shapes are the ragged ones: expert groups of 1, 127, 129 and 0 rows (the GEMM
computes whole 128-row tiles and relies on masks to drop the rows of the next expert), M = 1, and
an output width of 384 (a 256-column tile whose second half does not exist)."""
import numpy as np
import pytest
import torch

from paper_2604_07853_b200 import binding, build, inputs
from util import bits_to_torch

pytestmark = pytest.mark.gpu

POISON = 0xA5
GUARD = 1 << 16  # bytes of poison on each side


class Guarded:
    """A device buffer of `nbytes` usable bytes with GUARD poisoned bytes before and after."""

    def __init__(self, nbytes: int, dev):
        self.n = (nbytes + 255) // 256 * 256
        self.raw = torch.full((self.n + 2 * GUARD + 256,), POISON, dtype=torch.uint8, device=dev)
        base = self.raw.data_ptr()
        self.lo = (-(base + GUARD)) % 256 + GUARD          # usable part starts 256-byte aligned
        self.view = self.raw[self.lo:self.lo + self.n]
        self.exact = nbytes

    def check(self, what: str):
        torch.cuda.synchronize()
        before = self.raw[:self.lo]
        after = self.raw[self.lo + self.exact:]            # includes the rounding slack
        assert bool((before == POISON).all()), f"{what}: bytes before the buffer were written"
        assert bool((after == POISON).all()), f"{what}: bytes after the buffer were written"


@pytest.fixture(scope="module")
def ctx():
    build.build()
    c = binding.Context(0)
    yield c
    c.close()


@pytest.mark.parametrize("M,N,K", [(1, 128, 128), (1, 384, 256), (129, 384, 512), (127, 128, 1024), (300, 640, 256)])
def test_linear_leaves_surroundings_untouched(ctx, M, N, K):
    dev = torch.device("cuda", 0)
    case = inputs.linear_case(11, M, N, K)
    wc, ws = ctx.quantize_weight(bits_to_torch(case.w))
    x = bits_to_torch(case.x)
    ref = ctx.linear_fwd(x, wc, ws).clone()
    g_out = Guarded(M * N * 2, dev)
    g_ws = Guarded(int(ctx.lib.qarl_linear_workspace_bytes(M, N, K)), dev)
    out = g_out.view[:M * N * 2].view(torch.bfloat16).view(M, N)
    saved = ctx._ws
    ctx._ws = g_ws.view                                     # the call's workspace is the guarded slice
    try:
        y = ctx.linear_fwd(x, wc, ws, out=out)
    finally:
        ctx._ws = saved
    assert ctx.poll() == 0
    g_out.check("linear output")
    g_ws.check("linear workspace")
    assert torch.equal(y, ref)


def _grouped_ids(sizes, k=1):
    ids = np.concatenate([np.full(n, e, dtype=np.int32) for e, n in enumerate(sizes)])
    return ids.reshape(-1, k)


@pytest.mark.parametrize("sizes,H,I", [([1, 127, 129, 0], 384, 128), ([129, 0, 0, 1], 256, 256), ([0, 0, 0, 1], 384, 128),
                                       ([127, 1, 1, 127], 128, 128)])
def test_moe_leaves_surroundings_untouched(ctx, sizes, H, I):
    dev = torch.device("cuda", 0)
    E = len(sizes)
    ids_np = _grouped_ids(sizes)
    M = ids_np.shape[0]
    rng = np.random.default_rng(5)
    perm = rng.permutation(M)                               # tokens of a group are not contiguous in the batch
    ids_np = np.ascontiguousarray(ids_np[perm])
    c = inputs.moe_case(7, M, h=H, i=I, e=E, k=1)
    w13c, w13s = ctx.quantize_weight(bits_to_torch(c.w13))
    w2c, w2s = ctx.quantize_weight(bits_to_torch(c.w2))
    x = bits_to_torch(c.x)
    ids = torch.from_numpy(ids_np).to(dev)
    wts = torch.ones((M, 1), dtype=torch.float32, device=dev)
    ref = ctx.moe_fwd(x, ids, wts, w13c, w13s, w2c, w2s).clone()
    assert ctx.poll() == 0
    g_out = Guarded(M * H * 2, dev)
    g_ws = Guarded(ctx.moe_workspace_bytes(M, H, I, E, 1), dev)
    out = g_out.view[:M * H * 2].view(torch.bfloat16).view(M, H)
    y = ctx.moe_fwd(x, ids, wts, w13c, w13s, w2c, w2s, out=out, workspace=g_ws.view)
    assert ctx.poll() == 0
    g_out.check("moe output")
    g_ws.check("moe workspace")
    assert torch.equal(y, ref)
    # the dumps of the debug path are outputs too
    d_out = ctx.moe_fwd(x, ids, wts, w13c, w13s, w2c, w2s, debug=True)
    assert ctx.poll() == 0 and torch.equal(d_out[0], ref)


def test_bad_offsets_are_clamped_not_followed(ctx):
    """qarl_moe_experts_fwd takes caller-supplied group offsets: values past the row count or out of
    order must neither crash nor write outside the buffers; the status word reports them."""
    dev = torch.device("cuda", 0)
    E, H, I, R = 4, 256, 128, 200
    c = inputs.moe_case(9, R, h=H, i=I, e=E, k=1)
    w13c, w13s = ctx.quantize_weight(bits_to_torch(c.w13))
    w2c, w2s = ctx.quantize_weight(bits_to_torch(c.w2))
    xc, xs = ctx.quantize_act(bits_to_torch(c.x))
    pw = torch.ones(R, dtype=torch.float32, device=dev)
    g_out = Guarded(R * H * 2, dev)
    out = g_out.view[:R * H * 2].view(torch.bfloat16).view(R, H)
    for bad in ([0, 50, 100, 150, 100000], [0, 150, 50, 180, 200], [-7, 50, 100, 150, 200]):
        offs = torch.tensor(bad, dtype=torch.int32, device=dev)
        g_ws = Guarded(int(ctx.lib.qarl_moe_experts_workspace_bytes(R, I)), dev)
        saved = ctx._ws
        ctx._ws = g_ws.view
        try:
            ctx.moe_experts_fwd(xc, xs, pw, offs, w13c, w13s, w2c, w2s, out=out)
        finally:
            ctx._ws = saved
        assert ctx.poll() == -1                             # QARL_ERR_INVALID_ARG from the device
        g_out.check("experts output")
        g_ws.check("experts workspace")
