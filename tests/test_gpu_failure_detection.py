"""Failure detection without a GPU fault: a device-side wait that nothing satisfies gives up at
its limit, the kernel returns, the error is reported through the status word and the context keeps
working.  (The pipeline waits of the GEMM use the same bounded wait with a 2 s limit.)"""
import time

import numpy as np
import pytest
import torch

from paper_2604_07853_b200 import binding, build, inputs
from util import bits_to_torch

pytestmark = pytest.mark.gpu


def test_expired_wait_is_reported_and_context_survives():
    build.build()
    ctx = binding.Context(0)
    case = inputs.linear_case(3, 8, 128, 128)
    wc, ws = ctx.quantize_weight(bits_to_torch(case.w))
    before = ctx.linear_fwd(bits_to_torch(case.x), wc, ws).clone()
    assert ctx.poll() == 0
    t0 = time.perf_counter()
    ctx.harness_wait_selftest(limit_ns=2_000_000)          # 2 ms
    assert ctx.poll() == -7                                # QARL_ERR_DEVICE_TIMEOUT, then cleared
    assert time.perf_counter() - t0 < 1.0
    assert ctx.poll() == 0
    after = ctx.linear_fwd(bits_to_torch(case.x), wc, ws)  # the context is still usable
    assert torch.equal(before, after) and ctx.poll() == 0
    ctx.harness_wait_selftest(limit_ns=1000)
    with pytest.raises(binding.QarlError) as ei:
        ctx.check_device_status()
    assert ei.value.status == -7
    ctx.close()


@pytest.mark.parametrize("stop_after", [0, 1, 5])
def test_gemm_pipeline_wait_expires_and_context_survives(stop_after):
    """The FP8 GEMM's own abort protocol: the TMA producer stops arming stages (a host-set test
    switch), so the MMA role waits on a stage that nothing fills; its bounded wait (1 ms here)
    runs out, the CTA aborts, drains and frees its TMEM, the kernel returns, the status word says
    QARL_ERR_DEVICE_TIMEOUT, and the next call with the normal settings gives the reference bytes."""
    build.build()
    ctx = binding.Context(0)
    case = inputs.linear_case(5, 300, 384, 1024)           # 3 row tiles x 2 column tiles x 8 K-blocks
    wc, ws = ctx.quantize_weight(bits_to_torch(case.w))
    x = bits_to_torch(case.x)
    ref = ctx.linear_fwd(x, wc, ws).clone()
    assert ctx.poll() == 0
    ctx.harness_set_wait_limit_ns(1_000_000)
    ctx.harness_stop_producer_after(stop_after)
    t0 = time.perf_counter()
    ctx.linear_fwd(x, wc, ws)
    assert ctx.poll() == -7
    assert time.perf_counter() - t0 < 1.0
    ctx.harness_stop_producer_after(-1)
    ctx.harness_set_wait_limit_ns(0)
    assert ctx.poll() == 0
    for _ in range(2):
        assert torch.equal(ctx.linear_fwd(x, wc, ws), ref) and ctx.poll() == 0
    # the same through the grouped (MoE) kernels
    c = inputs.moe_case(2, 96, h=512, i=256, e=8, k=2)
    w13c, w13s = ctx.quantize_weight(bits_to_torch(c.w13))
    w2c, w2s = ctx.quantize_weight(bits_to_torch(c.w2))
    args = (bits_to_torch(c.x), torch.from_numpy(c.ids).cuda(), torch.from_numpy(c.weights).cuda(), w13c, w13s, w2c, w2s)
    ref_moe = ctx.moe_fwd(*args).clone()
    ctx.harness_set_wait_limit_ns(1_000_000)
    ctx.harness_stop_producer_after(min(stop_after, 2))     # a gate_up tile of this shape has 4 stages
    ctx.moe_fwd(*args)
    assert ctx.poll() == -7
    ctx.harness_stop_producer_after(-1)
    ctx.harness_set_wait_limit_ns(0)
    assert torch.equal(ctx.moe_fwd(*args), ref_moe) and ctx.poll() == 0
    ctx.close()


@pytest.mark.parametrize("stop_after", [0, 1, 5])
def test_router_pipeline_wait_expires_and_context_survives(stop_after):
    """The same for the one-launch router: its TMA producer stops arming stages, the MMA role's bounded
    wait (1 ms here) runs out, the CTA aborts (epilogue warps leave through the abort flag, logits
    stores in flight are waited for, TMEM is freed), the status word says QARL_ERR_DEVICE_TIMEOUT and
    the next call gives the reference bytes."""
    build.build()
    ctx = binding.Context(0)
    rng = np.random.default_rng(8)
    x = bits_to_torch(inputs.act_bf16(rng, 300, 512))       # 3 tiles of 8 contraction steps each
    wr = bits_to_torch(inputs.weight_bf16(rng, 64, 512))
    ref = [t.clone() for t in ctx.router_fwd(x, wr, 4)]
    assert ctx.poll() == 0
    ctx.harness_set_wait_limit_ns(1_000_000)
    ctx.harness_stop_producer_after(stop_after)
    t0 = time.perf_counter()
    ctx.router_fwd(x, wr, 4)
    assert ctx.poll() == -7
    assert time.perf_counter() - t0 < 1.0
    ctx.harness_stop_producer_after(-1)
    ctx.harness_set_wait_limit_ns(0)
    assert ctx.poll() == 0
    for _ in range(2):
        out = ctx.router_fwd(x, wr, 4)
        assert all(torch.equal(a.view(torch.int32), b.view(torch.int32)) for a, b in zip(out, ref)) and ctx.poll() == 0
    ctx.close()
