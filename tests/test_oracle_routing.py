"""Pins for the oracle's routing (logits, scoring, top-k, weights).  CPU only."""
import os

import numpy as np
import pytest
import torch

import oracle
from tests import oracle_twin as twin

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _bf16(x):
    return torch.tensor(np.asarray(x, np.float32)).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)


def _dummy_weights(E, H, I, g):
    return (np.full((E, 2 * I, H), 0x38, np.uint8), np.ones((E, 2 * I // g, H // g), np.float32),
            np.full((E, H, I), 0x38, np.uint8), np.ones((E, H // g, I // g), np.float32))


def _route(logit_rows, bias, K, scoring, renorm, routed_scale=1.0):
    """Build hidden = e_0 (one-hot) and Wr[e,0] = logit so that logits are exactly the given values."""
    E, H, g = len(logit_rows), 4, 4
    hidden = np.zeros((1, H), np.float32); hidden[0, 0] = 1.0
    Wr = np.zeros((E, H), np.float32); Wr[:, 0] = logit_rows
    r = oracle.moe_forward(_bf16(hidden), _bf16(Wr), None if bias is None else np.asarray(bias, np.float32),
                           *_dummy_weights(E, H, 4, g), top_k=K, scoring=scoring, renorm=renorm,
                           routed_scale=routed_scale, group=g)
    return r


def _gold():
    d = {}
    for line in open(os.path.join(GOLD, "routing_worked.txt")):
        if line.startswith("#") or not line.strip():
            continue
        kind, key, *vals = line.split()
        d[(kind, key)] = [float(v) for v in vals]
    return d


def test_softmax_worked_example_golden():
    g = _gold()
    r = _route(g[("softmax", "logits")], None, 1, oracle.SCORE_SOFTMAX, 1)
    assert r["ids"].tolist() == [[int(g[("softmax", "top1_id")][0])]] and r["w"][0, 0] == 1.0
    r = _route(g[("softmax", "logits")], None, 1, oracle.SCORE_SOFTMAX, 0)
    assert r["w"][0, 0] == np.float32(g[("softmax", "top1_w_raw")][0])
    r = _route(g[("softmax", "logits")], None, 2, oracle.SCORE_SOFTMAX, 1)
    assert r["ids"].tolist() == [[0, 1]]
    assert np.array_equal(r["w"][0], np.float32(g[("softmax", "top2_w")]))
    assert np.isinf(r["margin"][0])
    np.testing.assert_array_equal(r["logits"][0], np.float32(g[("softmax", "logits")]))


def test_sigmoid_bias_worked_example_golden():
    g = _gold()
    r = _route(g[("sigmoid", "logits")], g[("sigmoid", "bias")], 2, oracle.SCORE_SIGMOID_BIAS, 1)
    assert r["ids"].tolist() == [[int(v) for v in g[("sigmoid", "ids")]]]
    assert np.array_equal(r["w"][0], np.float32(g[("sigmoid", "w_renorm")]))
    keys = np.array(g[("sigmoid", "keys")])
    assert r["margin"][0] == pytest.approx(keys[1] - keys[3], abs=2e-8)   # bias is fp32: 0.3f, 0.6f
    r = _route(g[("sigmoid", "logits")], g[("sigmoid", "bias")], 2, oracle.SCORE_SIGMOID_BIAS, 0)
    assert np.array_equal(r["w"][0], np.float32(g[("sigmoid", "w_raw")]))
    # routed scaling factor multiplies the weights (Section 4.1: 2.5 for the sigmoid policies)
    r = _route(g[("sigmoid", "logits")], g[("sigmoid", "bias")], 2, oracle.SCORE_SIGMOID_BIAS, 1, routed_scale=2.5)
    np.testing.assert_allclose(r["w"][0], 2.5 * np.array(g[("sigmoid", "w_renorm")]), rtol=1e-7)
    # without the bias the selection follows the sigmoid itself: experts 0 and 3
    r = _route(g[("sigmoid", "logits")], None, 2, oracle.SCORE_SIGMOID_BIAS, 1)
    assert r["ids"].tolist() == [[0, 3]]


def test_ties_go_to_lowest_index_and_zero_hidden():
    r = _route([0.5, 1.0, 1.0, 1.0, 0.25], None, 2, oracle.SCORE_SOFTMAX, 1)
    assert r["ids"].tolist() == [[1, 2]] and r["w"][0].tolist() == [0.5, 0.5] and r["margin"][0] == 0.0
    r = _route([0.0] * 6, None, 3, oracle.SCORE_SOFTMAX, 1)
    assert r["ids"].tolist() == [[0, 1, 2]]
    np.testing.assert_allclose(r["w"][0], [1 / 3] * 3, rtol=1e-7)
    r = _route([0.0] * 6, [0, 0, 0.1, 0, 0.1, 0], 3, oracle.SCORE_SIGMOID_BIAS, 1)
    assert r["ids"].tolist() == [[2, 4, 0]]


@pytest.mark.parametrize("scoring", [0, 1])
@pytest.mark.parametrize("renorm", [0, 1])
def test_routing_matches_float64_argsort(scoring, renorm):
    rng = np.random.default_rng(10 + scoring * 2 + renorm)
    T, H, E, K, g = 7, 32, 24, 5, 4
    hidden = _bf16(rng.standard_normal((T, H)))
    Wr = _bf16(rng.standard_normal((E, H)) / np.sqrt(H))
    bias = (rng.standard_normal(E) * 0.1).astype(np.float32) if scoring else None
    r = oracle.moe_forward(hidden, Wr, bias, *_dummy_weights(E, H, 8, g), top_k=K, scoring=scoring,
                           renorm=renorm, group=g)
    ids, w, L = twin.route(hidden, Wr, bias, K, scoring, renorm)
    assert np.array_equal(r["ids"], ids)
    np.testing.assert_allclose(r["w"], w, rtol=2e-7)
    np.testing.assert_allclose(r["logits"], L, rtol=1e-6, atol=1e-7)
    for t in range(T):
        assert len(set(r["ids"][t])) == K
    if renorm:
        np.testing.assert_allclose(r["w"].sum(axis=1), 1.0, rtol=1e-6)
    assert (r["margin"] >= 0).all()


def test_top_k_equals_E_selects_everyone_in_key_order():
    rng = np.random.default_rng(5)
    E = 6
    logits = rng.standard_normal(E).astype(np.float32)
    logits = torch.tensor(logits).to(torch.bfloat16).to(torch.float32).numpy()
    r = _route(list(logits), None, E, oracle.SCORE_SOFTMAX, 1)
    assert r["ids"][0].tolist() == list(np.argsort(-logits, kind="stable"))
    p = np.exp(logits.astype(np.float64)); p /= p.sum()
    np.testing.assert_allclose(r["w"][0], p[r["ids"][0]], rtol=2e-7)
