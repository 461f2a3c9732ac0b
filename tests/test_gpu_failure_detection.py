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
