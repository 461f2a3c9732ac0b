"""Pins for the oracle's TBPO surrogate (Sec. 3.2: sequence-level ratio r_seq-prox and mismatch weight
w_seq-mismatch as geometric means of token ratios, two-sided TIS cap, sign-dependent bands, J = w~ r~ A)."""
import os

import numpy as np

import oracle

GOLD = os.path.join(os.path.dirname(__file__), "golden", "tbpo_paper_values.txt")


def _gold():
    ratios, consts = [], {}
    for line in open(GOLD):
        f = line.split()
        if not f or f[0].startswith("#"):
            continue
        if f[0] == "ratio":
            ratios.append(tuple(float(v) for v in f[1:]))
        else:
            consts[f[0]] = float(f[1])
    return ratios, consts


def _one(lp_cur, lp_old, lp_smp, adv, **kw):
    """A single response."""
    n = len(lp_cur)
    return oracle.tbpo(np.float32(lp_cur), np.float32(lp_old), np.float32(lp_smp), np.array([0, n]), np.float32([adv]), **kw)


def test_paper_worked_ratios_and_table_constants():
    ratios, consts = _gold()
    for p_old, p_new, printed in ratios:
        out = _one([np.log(p_new)], [np.log(p_old)], [np.log(p_old)], 1.0)
        assert abs(out["r"][0] - p_new / p_old) < 1e-6            # a one-token response: the token ratio itself
        assert abs(out["r"][0] - printed) < 0.011                 # as printed (two decimals / exact 2.5)
    d = oracle.TBPO_DEFAULTS
    assert d["eps_h"] == consts["seq_clip_ratio_high"] and d["delta_h"] == consts["neg_seq_clip_ratio_high"]
    assert d["delta_l"] == consts["neg_seq_clip_ratio_low"] and d["cap"] == consts["seq_tis_imp_ratio_cap"]


def test_identical_policies_give_the_plain_advantage():
    rng = np.random.default_rng(0)
    lens = [5, 1, 33, 7]
    off = np.concatenate([[0], np.cumsum(lens)])
    lp = rng.uniform(-5, -0.1, size=off[-1]).astype(np.float32)
    adv = np.float32([1.5, -0.5, 0.25, -2.0])
    out = oracle.tbpo(lp, lp, lp, off, adv)
    assert np.array_equal(out["r"], np.ones(4)) and np.array_equal(out["w"], np.ones(4))
    assert np.array_equal(out["J"], adv.astype(np.float64)) and (out["flags"] == 0).all()
    assert out["loss"] == -float(adv.astype(np.float64).mean())
    # gradient of -mean(J) w.r.t. each current-learner token log-prob: -A_i / (L_i B)
    for i, L in enumerate(lens):
        assert np.allclose(out["grad"][off[i]:off[i + 1]], -adv[i] / (L * 4), rtol=1e-7)


def test_geometric_mean_over_the_response():
    """r is exp(mean token log-ratio): constant per-token shift d gives exp(d) for any length, token
    order does not matter, and repeating the response's tokens leaves it unchanged."""
    rng = np.random.default_rng(1)
    old = rng.uniform(-4, -0.5, size=12)
    d = rng.normal(0, 1e-4, size=12)
    base = _one(old + d, old, old, 1.0)["r"][0]
    assert abs(base - np.exp(np.float32(old + d).astype(np.float64) - np.float32(old).astype(np.float64)).prod() ** (1 / 12)) < 1e-12
    perm = rng.permutation(12)
    assert abs(_one((old + d)[perm], old[perm], old[perm], 1.0)["r"][0] - base) < 1e-13
    assert abs(_one(np.tile(old + d, 3), np.tile(old, 3), np.tile(old, 3), 1.0)["r"][0] - base) < 1e-13
    # exactly representable shift: every token log-prob lower by 2^-12 -> r = exp(-2^-12) at any length
    for L in (1, 7, 4096):
        lp = np.full(L, -1.0)
        assert abs(_one(lp - 2.0 ** -12, lp, lp, 1.0)["r"][0] - np.exp(-2.0 ** -12)) < 1e-15


def test_tis_cap_is_two_sided_in_the_log_domain():
    lp = np.full(8, -2.0)
    for shift, expect_w, expect_cap, capped in [(0.5, np.exp(0.5), np.exp(0.5), False),
                                                (np.log(4.0), 4.0, 2.0, True),
                                                (-np.log(4.0), 0.25, 0.5, True),
                                                (-0.25, np.exp(-0.25), np.exp(-0.25), False)]:
        out = _one(lp, lp, lp - shift, 1.0)       # old learner vs old sampler differ by `shift` per token
        assert abs(out["w"][0] - expect_w) < 1e-6 * expect_w
        assert abs(out["J"][0] - expect_cap) < 1e-6 * expect_cap     # r = 1, A = 1: J = w~
        assert bool(out["flags"][0] & 2) == capped


def test_sign_dependent_bands_and_masking():
    lp = np.full(16, -1.0)
    eh, dl, dh = 4e-4, 3e-4, 7e-4
    cases = [  # (per-token log shift of the current learner, A, clipped?, r~)
        (np.log1p(2e-4), 1.0, False, None),        # inside [0, 1 + eps_h]
        (np.log1p(6e-4), 1.0, True, 1 + eh),       # above the positive band
        (np.log(0.5), 1.0, False, None),           # positive advantages have no lower bound but 0
        (np.log1p(6e-4), -1.0, False, None),       # inside [1 - dl, 1 + dh]: wider on top for A < 0
        (np.log1p(9e-4), -1.0, True, 1 + dh),      # dual clip: upper bound for negative samples
        (np.log1p(-5e-4), -1.0, True, 1 - dl),     # below the negative band
        (np.log1p(-2e-4), -1.0, False, None),
    ]
    for shift, A, clipped, rt in cases:
        out = _one(lp + shift, lp, lp, A)
        r = out["r"][0]
        assert abs(r - np.exp(np.float64(np.float32(-1.0 + shift)) + 1.0)) < 1e-12
        assert bool(out["flags"][0] & 1) == clipped
        assert abs(out["J"][0] - (rt if clipped else r) * A) < 1e-12
        if clipped:
            assert (out["grad"] == 0).all()        # the whole response is masked from the update
        else:
            assert np.allclose(out["grad"], -A * r / 16, rtol=1e-6)


def test_gradient_is_the_derivative_of_the_loss():
    rng = np.random.default_rng(2)
    lens = [3, 9, 4, 6, 2]
    off = np.concatenate([[0], np.cumsum(lens)])
    T = off[-1]
    old = rng.uniform(-3, -0.2, size=T).astype(np.float32)
    smp = (old + rng.normal(0, 0.05, size=T)).astype(np.float32)
    cur = (old + rng.normal(0, 2e-4, size=T)).astype(np.float32)
    adv = np.float32([1.0, -1.0, 0.5, -0.3, 2.0])
    out = oracle.tbpo(cur, old, smp, off, adv)
    h = np.float32(2.0 ** -10)
    for t in [0, 4, 13, 20, T - 1]:
        up, dn = cur.copy(), cur.copy()
        up[t] += h
        dn[t] -= h
        # a wide band so the finite difference does not cross a clip boundary
        kw = dict(eps_h=1.0, delta_l=0.9, delta_h=1.0)
        fd = (oracle.tbpo(up, old, smp, off, adv, **kw)["loss"] - oracle.tbpo(dn, old, smp, off, adv, **kw)["loss"]) / (2 * float(h))
        g = oracle.tbpo(cur, old, smp, off, adv, **kw)["grad"][t]
        assert abs(fd - g) < 1e-5 * max(1.0, abs(g))


def test_empty_response_and_mean_over_batch():
    lp = np.float32([-1.0, -1.0])
    out = oracle.tbpo(lp, lp, lp, np.array([0, 0, 2]), np.float32([3.0, 1.0]))
    assert out["flags"][0] == 4 and out["J"][0] == 0.0 and out["J"][1] == 1.0
    assert out["loss"] == -0.5                      # the empty response still counts in B
