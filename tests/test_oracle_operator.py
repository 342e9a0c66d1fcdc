"""Pins for the oracle's expert path and the whole operator.  CPU only.

Hand-worked 1-token case (tests/golden/hand_one_token.txt), dense float64
re-evaluation on tiny shapes (tests/oracle_twin.py), and invariants that any
correct implementation of the operator must satisfy.
"""
import os

import numpy as np
import pytest
import torch

import oracle
from paper_2609_04244_b200 import workloads as wl
from tests import oracle_twin as twin

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _bf16(x):
    return torch.tensor(np.asarray(x, np.float32)).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)


def _rand_problem(rng, T, H, E, I, g, scoring=0):
    hidden = _bf16(rng.standard_normal((T, H)))
    Wr = _bf16(rng.standard_normal((E, H)) / np.sqrt(H))
    bias = (rng.standard_normal(E) * 0.1).astype(np.float32) if scoring else None

    def codes(shape):  # random finite E4M3 codes with |value| <= 448, realistic spread
        c = rng.integers(0, 0x7F, size=shape, dtype=np.uint8)
        return c | (rng.integers(0, 2, size=shape, dtype=np.uint8) << 7)

    W13q, W2q = codes((E, 2 * I, H)), codes((E, H, I))
    W13s = rng.uniform(0.5, 2.0, (E, 2 * I // g, H // g)).astype(np.float32) * 2e-4
    W2s = rng.uniform(0.5, 2.0, (E, H // g, I // g)).astype(np.float32) * 2e-4
    return hidden, Wr, bias, W13q, W13s, W2q, W2s


def _gold_one_token():
    d = {}
    for line in open(os.path.join(GOLD, "hand_one_token.txt")):
        if line.startswith("#") or not line.strip():
            continue
        k, v = line.split()
        d[k] = v
    return d


def _hand_problem(w2_scale=2.0 ** -7, wr1=0.0, second=None):
    H = I = 128
    hidden = _bf16(np.ones((1, H)))
    Wr = np.zeros((2, H), np.float32); Wr[0] = 2.0 ** -7; Wr[1] = wr1
    W13q = np.full((2, 2 * I, H), 0x38, np.uint8); W2q = np.full((2, H, I), 0x38, np.uint8)
    W13s = np.zeros((2, 2, 1), np.float32); W13s[:, 0] = 2.0 ** -7; W13s[:, 1] = 2.0 ** -6
    W2s = np.full((2, 1, 1), w2_scale, np.float32)
    if second is not None:
        W13s[1] *= second
    return hidden, _bf16(Wr), None, W13q, W13s, W2q, W2s


def test_hand_worked_one_token_golden():
    g = _gold_one_token()
    r = oracle.moe_forward(*_hand_problem(), top_k=1)
    assert r["ids"].tolist() == [[0]] and r["w"][0, 0] == 1.0
    assert (r["xq"] == 0x7E).all() and r["xs"][0, 0] == np.float32(float(g["xs"]))
    assert (r["hq"] == 0x7E).all()
    assert np.allclose(r["act"], np.float32(float(g["a_fp32"])), rtol=0, atol=1.5e-7)
    assert (r["out"] == int(g["out_bf16_hex"], 16)).all()
    assert oracle.bf16_bits_to_f64(r["out"])[0, 0] == float(g["out_value"])
    # gate/up cross-check through the slot outputs: y = 448*hs
    np.testing.assert_allclose(r["out_f64"], 448.0 * float(r["hs"][0, 0]), rtol=1e-15)
    # power-of-two W2 scale -> output scales exactly
    r4 = oracle.moe_forward(*_hand_problem(w2_scale=2.0 ** -5), top_k=1)
    assert (r4["out"] == int(g["variant_w2scale_2^-5_out_hex"], 16)).all()
    # both experts identical, K = 2: same answer (weights sum to one)
    r2 = oracle.moe_forward(*_hand_problem(), top_k=2)
    assert r2["ids"].tolist() == [[0, 1]] and (r2["out"] == r["out"]).all()
    # router prefers expert 1, whose gate/up scales are halved: gate 0.5, up 1 -> a = silu(0.5)
    r1 = oracle.moe_forward(*_hand_problem(wr1=2.0 ** -6, second=0.5), top_k=1)
    assert r1["ids"].tolist() == [[1]]
    want = 0.5 / (1 + np.exp(-0.5))
    assert abs(oracle.bf16_bits_to_f64(r1["out"])[0, 0] - want) <= want * 2.0 ** -8 * 1.01


@pytest.mark.parametrize("T,H,E,I,K,g,scoring", [
    (1, 8, 2, 8, 1, 4, 0), (3, 16, 4, 8, 2, 4, 0), (5, 16, 5, 12, 5, 4, 1), (2, 256, 4, 128, 2, 128, 0),
    (4, 24, 6, 16, 3, 8, 1)])
def test_matches_dense_float64_twin(T, H, E, I, K, g, scoring):
    rng = np.random.default_rng(100 + T * 7 + H)
    prob = _rand_problem(rng, T, H, E, I, g, scoring)
    r = oracle.moe_forward(*prob, top_k=K, scoring=scoring, renorm=1, group=g, want_slots=True)
    tw = twin.forward(*prob, K=K, scoring=scoring, renorm=1, group=g)
    assert np.array_equal(r["ids"], tw["ids"])
    assert np.array_equal(r["xq"], tw["xq"]) and np.array_equal(r["xs"], tw["xs"])
    # SwiGLU output before requantisation: the two routes differ only in double rounding order
    a_or, a_tw = r["act"].reshape(T, K, I), tw["act"]
    np.testing.assert_allclose(a_or, a_tw, rtol=3e-7, atol=1e-30)
    same = np.array_equal(a_or, a_tw)
    if same:
        assert np.array_equal(r["hq"].reshape(T, K, I), tw["hq"])
        assert np.array_equal(r["hs"].reshape(T, K, -1), tw["hs"])
        np.testing.assert_allclose(r["y_slots"], tw["y"], rtol=1e-11, atol=1e-300)
        np.testing.assert_allclose(r["out_f64"], tw["out_f64"], rtol=1e-10, atol=1e-300)
    else:  # a 1-ulp fp32 difference in `a` may flip a code: compare through the oracle's own act
        mism = (r["hq"].reshape(T, K, I) != tw["hq"]).mean()
        assert mism < 0.02


def test_gate_is_first_half_up_is_second_half():
    """Swapping the halves of W13 must change the result (silu(g)*u is not symmetric)."""
    rng = np.random.default_rng(7)
    hidden, Wr, bias, W13q, W13s, W2q, W2s = _rand_problem(rng, 2, 16, 3, 8, 4)
    r = oracle.moe_forward(hidden, Wr, bias, W13q, W13s, W2q, W2s, top_k=2, group=4)
    sw_q = np.concatenate([W13q[:, 8:], W13q[:, :8]], axis=1)
    sw_s = np.concatenate([W13s[:, 2:], W13s[:, :2]], axis=1)
    r2 = oracle.moe_forward(hidden, Wr, bias, sw_q, sw_s, W2q, W2s, top_k=2, group=4)
    assert not np.allclose(r["out_f64"], r2["out_f64"])
    tw = twin.forward(hidden, Wr, bias, W13q, W13s, W2q, W2s, K=2, scoring=0, renorm=1, group=4)
    gate = tw["g"][..., :8]
    np.testing.assert_allclose(r["act"].reshape(2, 2, 8), gate / (1 + np.exp(-gate)) * tw["g"][..., 8:], rtol=3e-7)


def _c1_like(T, seed=0, scoring=0, E=6, K=2):
    shape = wl.MoEShape("t", 1, H=256, E=E, I=128, top_k=K, scoring=scoring)
    d = wl.make_layer(shape, T, layer=seed)
    hid = d["hidden"].view(torch.int16).numpy().view(np.uint16)
    Wr = d["Wr"].view(torch.int16).numpy().view(np.uint16)
    bias = None if d["bias"] is None else d["bias"].numpy()
    return shape, [hid, Wr, bias, d["W13q"].numpy(), d["W13s"].numpy(), d["W2q"].numpy(), d["W2s"].numpy()]


def test_invariant_identical_experts_output_independent_of_routing():
    shape, p = _c1_like(3)
    for k in (3, 4, 5, 6):
        p[k] = np.repeat(p[k][:1], shape.E, axis=0)
    base = oracle.moe_forward(*p, top_k=1)
    for K in (2, 4):
        r = oracle.moe_forward(*p, top_k=K, want_slots=True)
        for j in range(1, K):
            assert np.array_equal(r["y_slots"][:, j], r["y_slots"][:, 0])
        np.testing.assert_allclose(r["out_f64"], base["out_f64"], rtol=1e-6)
    r0 = oracle.moe_forward(*p, top_k=3, renorm=0)
    np.testing.assert_allclose(r0["out_f64"], base["out_f64"] * r0["w"].astype(np.float64).sum(1, keepdims=True),
                               rtol=1e-6)
    p2 = list(p); p2[1] = p[1][::-1].copy()   # a different router: same output
    assert np.array_equal(oracle.moe_forward(*p2, top_k=2)["out"], oracle.moe_forward(*p, top_k=2)["out"])


def test_invariant_topk_equals_E_is_dense_mixture():
    shape, p = _c1_like(2, seed=1, E=4)
    r = oracle.moe_forward(*p, top_k=4, renorm=1, want_slots=True)
    r0 = oracle.moe_forward(*p, top_k=4, renorm=0)
    np.testing.assert_allclose(r["w"], r0["w"], rtol=3e-7)           # renormalising a full softmax is a no-op
    L = twin.bf16_bits_to_f64(p[0]) @ twin.bf16_bits_to_f64(p[1]).T
    P = np.exp(L - L.max(1, keepdims=True)); P /= P.sum(1, keepdims=True)
    dense = np.zeros_like(r["out_f64"])
    for e in range(4):
        single = oracle.moe_forward(*p, top_k=1, ids_in=np.full((2, 1), e), w_in=np.ones((2, 1)))
        dense += P[:, e:e + 1] * single["out_f64"]
    np.testing.assert_allclose(r["out_f64"], dense, rtol=1e-6, atol=1e-7 * np.abs(dense).max())


def test_invariant_power_of_two_scaling():
    shape, p = _c1_like(2, seed=2)
    r = oracle.moe_forward(*p, top_k=2)
    p2 = list(p); p2[6] = p[6] * np.float32(4.0)
    r2 = oracle.moe_forward(*p2, top_k=2)
    assert np.array_equal(r2["out_f64"], r["out_f64"] * 4.0)
    # hidden * 2^k on the expert path (routing held fixed): identical codes, scales * 2^k
    h2 = _bf16(oracle.bf16_bits_to_f64(p[0]) * 8.0)
    r3 = oracle.moe_forward(h2, *p[1:], top_k=2, ids_in=r["ids"], w_in=r["w"])
    assert np.array_equal(r3["xq"], r["xq"]) and np.array_equal(r3["xs"], r["xs"] * np.float32(8))


def test_invariant_per_token_independence_and_zero_hidden():
    shape, p = _c1_like(5, seed=3)
    r = oracle.moe_forward(*p, top_k=2)
    for t in (0, 3):
        rt = oracle.moe_forward(p[0][t:t + 1], *p[1:], top_k=2)
        assert np.array_equal(rt["out"][0], r["out"][t]) and np.array_equal(rt["ids"][0], r["ids"][t])
        assert np.array_equal(rt["xq"][0], r["xq"][t])
    z = oracle.moe_forward(np.zeros_like(p[0]), *p[1:], top_k=2)
    assert not z["out"].any() and z["ids"].tolist() == [[0, 1]] * 5


def test_invariant_expert_permutation():
    shape, p = _c1_like(3, seed=4, scoring=1)
    perm = np.array([3, 0, 5, 1, 4, 2])
    q = [p[0], p[1][perm], p[2][perm]] + [a[perm] for a in p[3:]]
    r = oracle.moe_forward(*p, top_k=2, scoring=1)
    rp = oracle.moe_forward(*q, top_k=2, scoring=1)
    assert np.array_equal(perm[rp["ids"]], r["ids"])
    assert np.array_equal(rp["out"], r["out"])


def test_compacted_expert_map_gives_identical_result():
    shape, p = _c1_like(3, seed=5)
    r = oracle.moe_forward(*p, top_k=2)
    used = np.unique(r["ids"])
    emap = np.full(shape.E, -1, np.int32); emap[used] = np.arange(len(used))
    rc = oracle.moe_forward(p[0], p[1], p[2], p[3][used], p[4][used], p[5][used], p[6][used], top_k=2,
                            expert_map=emap)
    assert np.array_equal(rc["out"], r["out"])


@pytest.mark.parametrize("dist", ["gauss", "student_t3"])
def test_quantisation_error_sanity_cosine(dist):
    """Section 4.2: cosine similarity against an unquantised evaluation stays >= 0.998 with routing held fixed."""
    shape = wl.MoEShape("t", 1, H=512, E=4, I=256, top_k=2, scoring=0)
    g = torch.Generator().manual_seed(11)

    def draw(*s):
        if dist == "gauss":
            x = torch.randn(*s, generator=g)
        else:
            x = torch.randn(*s, generator=g) / (torch.randn(3, *s, generator=g).square().sum(0) / 3).sqrt()
        return x / x.square().mean().sqrt()

    for T in (1, 4):
        X = draw(T, shape.H)
        W13 = draw(shape.E, 2 * shape.I, shape.H) * 0.02
        W2 = draw(shape.E, shape.H, shape.I) * 0.02
        q13 = [wl.pack_fp8_blockwise(W13[e]) for e in range(shape.E)]
        q2 = [wl.pack_fp8_blockwise(W2[e]) for e in range(shape.E)]
        ids = np.stack([np.arange(2) + (t % 3) for t in range(T)]).astype(np.int32)
        w = np.full((T, 2), 0.5, np.float32)
        hid = X.to(torch.bfloat16)
        r = oracle.moe_forward(hid.view(torch.int16).numpy().view(np.uint16), np.zeros((shape.E, shape.H), np.uint16),
                               None, np.stack([a[0].numpy() for a in q13]), np.stack([a[1].numpy() for a in q13]),
                               np.stack([a[0].numpy() for a in q2]), np.stack([a[1].numpy() for a in q2]),
                               top_k=2, ids_in=ids, w_in=w)
        Xd = X.double()
        ref = torch.zeros(T, shape.H, dtype=torch.float64)
        for t in range(T):
            for j in range(2):
                gu = W13[ids[t, j]].double() @ Xd[t]
                a = torch.nn.functional.silu(gu[:shape.I]) * gu[shape.I:]
                ref[t] += 0.5 * (W2[ids[t, j]].double() @ a)
        got = torch.from_numpy(r["out_f64"])
        cos = torch.nn.functional.cosine_similarity(got.flatten(), ref.flatten(), dim=0).item()
        assert cos >= 0.998, cos
