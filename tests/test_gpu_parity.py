"""GPU parity: the CUDA library (through its C ABI) against the CPU oracle.  Needs a B200."""
import numpy as np
import pytest
import torch

from paper_2609_04244_b200 import workloads as wl
from tests.parity import run_case

pytestmark = pytest.mark.gpu

TINY = wl.MoEShape("tiny", 1, H=256, E=8, I=128, top_k=2, scoring=wl.SCORE_SOFTMAX)
SMALL_SIG = wl.MoEShape("small_sig", 5, H=512, E=32, I=256, top_k=4, scoring=wl.SCORE_SIGMOID_BIAS)
RAGGED = wl.MoEShape("ragged", 2, H=384, E=20, I=640, top_k=3, scoring=wl.SCORE_SOFTMAX)


@pytest.mark.parametrize("T", [1, 2, 5, 9, 16, 17, 32, 33, 64])
def test_tiny_all_token_tiles(T):
    """Every kernel variant: token columns 1..8, tokens compacted per expert (9..32 here), all tokens as columns (33, 64)."""
    r = run_case(TINY, T, repeat=2)
    assert r["rel_l2"] < 2e-3, r


@pytest.mark.parametrize("shape,T", [(SMALL_SIG, 1), (SMALL_SIG, 8), (SMALL_SIG, 40), (RAGGED, 3), (RAGGED, 24)])
def test_small_shapes_sigmoid_and_ragged(shape, T):
    r = run_case(shape, T, repeat=2)
    assert r["rel_l2"] < 2e-3, r


def test_config1_tiny_moe():
    r = run_case(wl.SHAPES["c1_tiny"], 1, repeat=3)
    assert r["rel_l2"] < 2e-3 and r["unique_experts"] == 2, r


@pytest.mark.parametrize("T", [1, 8])
def test_config2_qwen3_like(T):
    r = run_case(wl.SHAPES["c2_qwen3_30b_a3b"], T, repeat=2)
    assert r["rel_l2"] < 2e-3, r


@pytest.mark.parametrize("regime,T", [("same", 4), ("disjoint", 4), ("disjoint", 32), ("natural", 64), ("same", 40), ("same", 64),
                                      ("natural", 128), ("same", 128)])
def test_config3_routing_regimes(regime, T):
    """Natural, maximum-reuse and maximum-bytes routing; 40 and 64 tokens on the same 8 experts walk each expert in
    three and four passes of 16 compacted tokens, 128 tokens in eight."""
    r = run_case(wl.SHAPES["c2_qwen3_30b_a3b"], T, regime=regime, max_oracle_tokens=8)
    if regime == "same":      # (at 128 tokens the forcing term of the generator no longer wins for every token)
        assert r["unique_experts"] == 8 if T <= 64 else r["unique_experts"] <= 16
    if regime == "disjoint":
        assert r["unique_experts"] == min(128, 8 * T)
    assert r["rel_l2"] < 2e-3, r


@pytest.mark.parametrize("weight,slack", [(0, 200), (4, 100), (8, 0), (4, 1 << 20)])
@pytest.mark.parametrize("shape,regime,T", [(SMALL_SIG, "natural", 12), (SMALL_SIG, "same", 40), (RAGGED, "natural", 24),
                                            (RAGGED, "same", 128), (wl.SHAPES["c2_qwen3_30b_a3b"], "same", 64),
                                            (wl.SHAPES["c2_qwen3_30b_a3b"], "natural", 33)])
def test_ranges_of_equal_weight(shape, regime, T, weight, slack):
    """Where tokens are compacted the per-CTA ranges are cut by weight (a k-step of a crowded expert weighs more), in
    both compacted variants, with units split across CTAs (slack 0) and kept whole (huge slack); weight 0 is the
    equal-length cut.  Every setting must match the oracle and repeat bit-identically."""
    r = run_case(shape, T, regime=regime, max_oracle_tokens=8, repeat=2, knobs={"split_weight": weight, "split_slack_kib": slack})
    assert r["rel_l2"] < 2e-3, r


@pytest.mark.parametrize("shape,per_launch", [(SMALL_SIG, 128), (TINY, 64)])
def test_more_tokens_than_one_launch_is_chunked(shape, per_launch):
    """More tokens than one launch takes (128 under sparse routing, else 64) run as consecutive launches; each chunk
    must match the oracle and the one-call result."""
    from paper_2609_04244_b200 import MoEPlan
    from tests.parity import check_against_oracle
    plan = MoEPlan(shape.H, shape.E, shape.I, shape.top_k, shape.scoring, shape.renorm, T_max=per_launch + 36)
    assert plan.tokens_per_launch() == per_launch
    T = per_launch + 36
    d = wl.make_layer(shape, T, device="cuda")
    args = (d["Wr"], d["bias"], d["W13q"], d["W13s"], d["W2q"], d["W2s"])
    full = plan.forward(d["hidden"], *args)
    plan.sync_status()
    for lo, hi in ((0, per_launch), (per_launch, T)):
        dbg = plan.forward_debug(d["hidden"][lo:hi].contiguous(), *args)
        plan.sync_status()
        assert torch.equal(dbg["out"], full[lo:hi])
        dd = dict(d, hidden=d["hidden"][lo:hi].contiguous())
        r = check_against_oracle(shape, hi - lo, dd, dbg, max_oracle_tokens=12)
        assert r["rel_l2"] < 2e-3, r
    plan.close()


@pytest.mark.parametrize("shape,T", [(SMALL_SIG, 128), (SMALL_SIG, 97), (RAGGED, 128)])
def test_up_to_128_tokens_in_one_launch(shape, T):
    """65..128 tokens in a single launch: token sets of two 64-bit words, up to eight passes of 16 compacted tokens."""
    r = run_case(shape, T)
    assert r["rel_l2"] < 2e-3, r


def test_host_activation_entry_point_matches_device_entry_point():
    """moe_forward_host stages pinned host activations through the workspace; same kernel, same bits."""
    from paper_2609_04244_b200 import MoEPlan
    shape, T = SMALL_SIG, 70                                   # > 64: two chunks through the staging area
    d = wl.make_layer(shape, T, device="cuda")
    plan = MoEPlan(shape.H, shape.E, shape.I, shape.top_k, shape.scoring, shape.renorm, T_max=T)
    args = (d["Wr"], d["bias"], d["W13q"], d["W13s"], d["W2q"], d["W2s"])
    ref = plan.forward(d["hidden"], *args)
    h_in = d["hidden"].cpu().pin_memory()
    h_out = torch.zeros((T, shape.H), dtype=torch.bfloat16).pin_memory()
    plan.forward_host(h_in, *args, h_out)
    plan.sync_status()
    assert torch.equal(h_out, ref.cpu())
    plan.close()


@pytest.mark.parametrize("name,T,pinned", [("c2_qwen3_30b_a3b", 1, True), ("c2_qwen3_30b_a3b", 1, False), ("c2_qwen3_30b_a3b", 3, True),
                                           ("c1_tiny", 1, True), ("small_sig", 1, True), ("small_sig", 8, True)])
def test_host_entry_point_small_token_counts(name, T, pinned):
    """Few tokens from host memory: the result is written by the kernel straight into a pinned output buffer; pageable
    buffers take the staged path.  Same bits as the device entry point either way, also when the host buffers change
    between calls."""
    from paper_2609_04244_b200 import MoEPlan
    shape = SMALL_SIG if name == "small_sig" else wl.SHAPES[name]
    plan = MoEPlan(shape.H, shape.E, shape.I, shape.top_k, shape.scoring, shape.renorm, T_max=T)
    for layer in range(3):
        d = wl.make_layer(shape, T, layer=layer, device="cuda")
        args = (d["Wr"], d["bias"], d["W13q"], d["W13s"], d["W2q"], d["W2s"])
        ref = plan.forward(d["hidden"], *args).clone()
        h_in = d["hidden"].cpu()
        h_out = torch.zeros((T, shape.H), dtype=torch.bfloat16)
        if pinned:
            h_in, h_out = h_in.pin_memory(), h_out.pin_memory()
        plan.forward_host(h_in, *args, h_out)
        plan.sync_status()
        assert torch.equal(h_out, ref.cpu()), (name, T, layer)
    plan.close()
