"""Pins for the oracle's router (top-k softmax over bf16 logits; ties to the lower expert id)."""
import numpy as np

import oracle
from paper_2604_07853_b200 import inputs


def test_hand_worked_token():
    """logits (0, ln 2, ln 4, -5) and k = 2: experts 2 then 1; softmax over (ln 4, ln 2) = (2/3, 1/3)."""
    l = np.float32([[0.0, np.log(2.0), np.log(4.0), -5.0]])
    ids, w = oracle.router_topk(l, 2)
    assert ids.tolist() == [[2, 1]]
    assert np.allclose(w, [[2 / 3, 1 / 3]], rtol=1e-6)


def test_ties_go_to_the_lower_id_and_order_is_descending():
    l = np.float32([[1.0, 3.0, 3.0, 2.0, 3.0, 0.0]])
    ids, w = oracle.router_topk(l, 4)
    assert ids.tolist() == [[1, 2, 4, 3]]
    assert np.allclose(w.sum(), 1.0, rtol=1e-6) and w[0, 0] == w[0, 1] == w[0, 2] > w[0, 3]
    ids, w = oracle.router_topk(np.zeros((1, 8), np.float32), 8)         # all equal: identity order, uniform weights
    assert ids.tolist() == [list(range(8))] and np.allclose(w, 1 / 8)


def test_against_the_input_generators_selection():
    """The seeded generator that draws routing for the other tests selects by an independent numpy
    argsort; on its logits the oracle's selection must agree."""
    rng = np.random.default_rng(0)
    M, E, k = 200, 128, 8
    logits = rng.normal(size=(M, E)).astype(np.float32)
    ids, w = oracle.router_topk(logits, k)
    order = np.argsort(-logits, axis=1, kind="stable")[:, :k]
    assert np.array_equal(ids, order)
    sel = np.take_along_axis(logits, order, axis=1).astype(np.float64)
    ref = np.exp(sel - sel[:, :1])
    ref /= ref.sum(axis=1, keepdims=True)
    assert np.allclose(w, ref, rtol=1e-6)
    assert np.allclose(w.astype(np.float64).sum(axis=1), 1.0, atol=1e-6)


def test_router_logits_are_the_bf16_linear():
    rng = np.random.default_rng(1)
    x = inputs.act_bf16(rng, 16, 256)
    wr = inputs.weight_bf16(rng, 32, 256)
    logits, ids, w = oracle.router(x, wr, 4)
    ref = inputs.bf16_bits_to_f32(x).astype(np.float64) @ inputs.bf16_bits_to_f32(wr).astype(np.float64).T
    assert np.array_equal(logits, ref.astype(np.float32))
    assert np.array_equal(ids[:, 0], logits.argmax(axis=1))
