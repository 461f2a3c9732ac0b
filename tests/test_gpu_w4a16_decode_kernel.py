"""The W4A16 / FP4A16 grouped GEMM has a wide-tile kernel (token rows on the MMA's M side) and a
swapped-operand kernel for decode-sized groups (expanded weight rows on the M side, at most 32
token rows on the N side).  Both must give the same bytes for every row (App. C: the fixed
K-reduction order holds across kernels): one input goes through both, forced by the harness
switch, and every stage the layer exposes is compared bit for bit; the automatic choice too."""
import pytest
import torch

from paper_2604_07853_b200 import binding, build, inputs
from test_gpu_w4a16 import DeviceCase, Int4
from test_gpu_fp4a16 import E2m1

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    build.build()
    c = binding.Context(0)
    yield c
    c.harness_set_gemm_path(0)
    c.close()


def _layer(ctx, dc, path, debug=True):
    ctx.harness_set_gemm_path(path)
    r = dc.run(ctx, debug=debug)
    assert ctx.poll() == 0
    ctx.harness_set_gemm_path(0)
    return r


@pytest.mark.parametrize("fmt", [Int4, E2m1])
@pytest.mark.parametrize("m,h,i,e,k,zipf", [(256, 2048, 768, 128, 8, None), (64, 512, 256, 8, 2, None), (1, 512, 256, 8, 2, None),
                                             (8, 2048, 768, 128, 8, None), (33, 256, 384, 2, 1, None),
                                             (300, 512, 256, 8, 2, 1.1), (100, 512, 128, 16, 4, 1.5)])
def test_decode_kernel_equals_wide_kernel_stage_by_stage(ctx, fmt, m, h, i, e, k, zipf):
    c = inputs.moe_case(31, m, h=h, i=i, e=e, k=k, zipf_s=zipf)
    dc = DeviceCase(ctx, c, fmt)
    out_w, d_w = _layer(ctx, dc, 1)
    for path in (2, 0):
        out_d, d_d = _layer(ctx, dc, path)
        for key in ("expert_offsets", "sorted_pair", "gate_up", "h", "down_f32"):
            assert torch.equal(d_w[key].view(torch.uint8), d_d[key].view(torch.uint8)), (path, key)
        assert torch.equal(out_w, out_d), path
    wide = _layer(ctx, dc, 1, debug=False).clone()
    assert torch.equal(wide, _layer(ctx, dc, 2, debug=False))
    assert torch.equal(wide, _layer(ctx, dc, 0, debug=False))
