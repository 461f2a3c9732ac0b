"""The allocation-free dense projection (qarl_linear_fwd_static) gives the same bytes as
qarl_linear_fwd.  It exists for callers that cannot obtain device memory at call time (a
server whose memory pool already owns the whole GPU, a plugin under someone else's allocator):
its scratch is a fixed array inside the library, shared by every call on the device and never
cleared.  Two calls in a row, the second on a smaller and different input, check that nothing
stale from the first call leaks into the second.  The test needs no state from any other test
(it creates its own context) and leaves none behind."""
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
    assert c.poll() == 0
    c.close()


def test_static_scratch_entry_point_matches_workspace_entry_point(ctx):
    first = inputs.linear_case(41, 300, 640, 1024)
    second = inputs.linear_case(42, 37, 384, 512)       # fewer rows, different K: stale data would show
    for case in (first, second):
        wc, ws = ctx.quantize_weight(bits_to_torch(case.w))
        x = bits_to_torch(case.x)
        want = ctx.linear_fwd(x, wc, ws).clone()
        out = torch.full((case.M, case.N), float("nan"), dtype=torch.bfloat16, device="cuda")
        got = ctx.linear_fwd_static(x, wc, ws, out)
        assert ctx.poll() == 0
        assert torch.equal(got, want)                   # same kernels, same order: bitwise equal
    # and once more on the first input, after the smaller call overwrote part of the scratch
    wc, ws = ctx.quantize_weight(bits_to_torch(first.w))
    x = bits_to_torch(first.x)
    out = torch.empty((first.M, first.N), dtype=torch.bfloat16, device="cuda")
    assert torch.equal(ctx.linear_fwd_static(x, wc, ws, out), ctx.linear_fwd(x, wc, ws))


def test_static_scratch_limit_is_enforced_with_a_clear_error(ctx):
    K = 2048
    M = binding.STATIC_LINEAR_MAX_ELEMS // K + 1
    x = torch.zeros((M, K), dtype=torch.bfloat16, device="cuda")
    wc = torch.zeros((128, K), dtype=torch.uint8, device="cuda")
    ws = torch.ones((1, K // 128), dtype=torch.float32, device="cuda")
    out = torch.empty((M, 128), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(binding.QarlError) as ei:
        ctx.linear_fwd_static(x, wc, ws, out)
    assert ei.value.status == -2 and "exceeds the built-in scratch" in str(ei.value)
    # exactly at the limit is accepted
    M = binding.STATIC_LINEAR_MAX_ELEMS // K
    ctx.linear_fwd_static(x[:M], wc, ws, out[:M])
    assert ctx.poll() == 0
