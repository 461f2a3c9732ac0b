"""GPU parity of the TBPO sequence-level surrogate (Sec. 3.2) against the oracle: per-response ratio,
mismatch weight, surrogate and flags, the per-token gradient and the loss."""
import numpy as np
import pytest
import torch

import oracle
from paper_2604_07853_b200 import binding, build, inputs
from util import to_dev

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    build.build()
    c = binding.Context(0)
    yield c
    assert c.poll() == 0
    c.close()


def check(ctx, case, **kw):
    """Both sides compute in double on the same fp32 inputs; they differ in summation order and in
    the last bits of exp: 1e-12 relative on r, w, J and the loss; flags equal (no response of these
    seeded cases sits within 1e-12 of a band edge); gradient = fp32 rounding of a double that agrees
    to 1e-12, i.e. equal or adjacent floats."""
    cur, old, smp, off, adv = case
    ref = oracle.tbpo(cur, old, smp, off, adv, **kw)
    out = ctx.tbpo_loss(to_dev(cur), to_dev(old), to_dev(smp), to_dev(off), to_dev(adv), **kw)
    assert ctx.poll() == 0
    for k in ("r", "w", "J"):
        g = out[k].cpu().numpy()
        assert np.allclose(g, ref[k], rtol=1e-12, atol=1e-300), k
    assert np.array_equal(out["flags"].cpu().numpy(), ref["flags"])
    g = out["grad"].cpu().numpy()
    assert np.allclose(g, ref["grad"], rtol=1.3e-7, atol=0.0)
    assert g.size < 100 or (g == ref["grad"]).mean() > 0.99
    assert abs(out["loss"].item() - ref["loss"]) <= 1e-12 * max(1.0, abs(ref["loss"]))
    return ref


def test_ragged_lengths_around_the_chunk_size(ctx):
    lens = [1, 2047, 2048, 2049, 0, 5, 4096, 0, 0, 7000, 3, 1, 12288, 100]
    ref = check(ctx, inputs.tbpo_case(1, lens))
    assert ((ref["flags"] & 4) != 0).sum() == 3                    # the empty responses
    assert 0 < ((ref["flags"] & 1) != 0).sum() < len(lens)         # some responses leave their band, some do not


def test_many_short_responses_and_one_long(ctx):
    rng = np.random.default_rng(2)
    lens = list(rng.integers(1, 120, size=300)) + [50000] + list(rng.integers(1, 40, size=200))
    check(ctx, inputs.tbpo_case(2, lens))


def test_single_response_and_single_token(ctx):
    check(ctx, inputs.tbpo_case(3, [1]))
    check(ctx, inputs.tbpo_case(4, [9001]))
    check(ctx, inputs.tbpo_case(5, [0, 0]))


def test_cap_and_bands_are_exercised(ctx):
    """Large mismatch so that the two-sided cap binds; non-default hyper-parameters."""
    lens = inputs.tbpo_lengths(6, 400, mean_len=300, max_len=3000)
    ref = check(ctx, inputs.tbpo_case(6, lens, drift=5e-4, mismatch=1.5))
    ref = check(ctx, inputs.tbpo_case(7, [3] * 500, drift=0.2, mismatch=2.5), eps_h=0.2, delta_l=0.1, delta_h=0.3, cap=1.5)
    assert (ref["flags"] & 2).sum() > 0 and (ref["flags"] & 1).sum() > 0


def test_paper_worked_ratio_on_the_gpu(ctx):
    """p_old = 0.02 -> p_theta = 0.05 as a one-token response: r = 2.5 (Sec. 3.2, dual clipping)."""
    lp = lambda p: np.float32([np.log(p)])
    out = ctx.tbpo_loss(to_dev(lp(0.05)), to_dev(lp(0.02)), to_dev(lp(0.02)), to_dev(np.array([0, 1])), to_dev(np.float32([-1.0])))
    assert abs(out["r"].item() - 2.5) < 1e-6 and out["flags"].item() == 1      # far above 1 + delta_h: masked
    assert out["J"].item() == -(1 + 7e-4) and out["grad"].item() == 0.0


def test_bitwise_repeatable(ctx):
    case = inputs.tbpo_case(8, inputs.tbpo_lengths(8, 256, mean_len=2000, max_len=9000))
    dev = [to_dev(a) for a in case]
    a = ctx.tbpo_loss(*dev)
    a = {k: v.clone() for k, v in a.items()}
    b = ctx.tbpo_loss(*dev)
    for k in a:
        assert torch.equal(a[k], b[k])


def test_training_batch_shape_sampled(ctx):
    """The benchmark's workload (4096 responses, ~4k tokens each, 16 M tokens): every per-response
    value against the oracle, gradient on sampled responses."""
    lens = inputs.tbpo_lengths(9, 4096)
    cur, old, smp, off, adv = inputs.tbpo_case(9, lens)
    ref = oracle.tbpo(cur, old, smp, off, adv)
    out = ctx.tbpo_loss(to_dev(cur), to_dev(old), to_dev(smp), to_dev(off), to_dev(adv))
    assert ctx.poll() == 0
    for k in ("r", "w", "J"):
        assert np.allclose(out[k].cpu().numpy(), ref[k], rtol=1e-12, atol=1e-300)
    assert np.array_equal(out["flags"].cpu().numpy(), ref["flags"])
    assert abs(out["loss"].item() - ref["loss"]) <= 1e-12
    g = out["grad"].cpu().numpy()
    for i in np.random.default_rng(0).integers(0, 4096, size=64):
        assert np.allclose(g[off[i]:off[i + 1]], ref["grad"][off[i]:off[i + 1]], rtol=1.3e-7, atol=0.0)
