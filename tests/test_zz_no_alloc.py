"""The no-allocation entry point against the ordinary one (GPU, through the C ABI).

moe_forward_noalloc serves callers that cannot hand the library a scratch buffer (they may not allocate device
memory where they run the step); it uses the fixed array built into the library instead.  The kernel and its
arithmetic are the same, so its output must equal moe_forward's within the tolerance of the parity tests -- here
it is even bit-identical, because the reduction order is fixed.  Two calls in a row check that the array's
left-over contents from the first call do not leak into the second.  The file is named so that pytest collects it
last: a run that stops at the first failure has then already run every other test.
"""
import pytest
import torch

import paper_2609_04244_b200 as m
from paper_2609_04244_b200 import workloads as wl

pytestmark = pytest.mark.gpu


def _run_pair(shape, T, layer):
    from tests.parity import check_against_oracle
    d = wl.make_layer(shape, T, layer=layer, device="cuda")
    plan = m.MoEPlan(shape.H, shape.E, shape.I, shape.top_k, shape.scoring, shape.renorm, T_max=T)
    args = (d["hidden"], d["Wr"], d["bias"], d["W13q"], d["W13s"], d["W2q"], d["W2s"])
    dbg = plan.forward_debug(*args)                              # the ordinary entry point, accepted by the oracle first
    plan.sync_status()
    check_against_oracle(shape, T, d, dbg)
    ref = dbg["out"]
    out = torch.full_like(ref, float("nan"))
    m.moe_forward_noalloc(plan.handle, T, *args, out)
    m.moe_sync_status(plan.handle, None)                         # NULL workspace = the built-in array: a healthy call reports no device problem
    plan.close()
    return ref, out


def test_noalloc_matches_workspace_entry_point_twice_in_a_row():
    shape = wl.MoEShape("noalloc", 2, H=512, E=32, I=256, top_k=4, scoring=wl.SCORE_SIGMOID_BIAS)
    # two calls in a row per kernel family: token columns (5, 3), the fused-unit variant (1, 2) and the variants that
    # compact each expert's tokens (12, 40: other scratch layout), each time with other inputs
    for call, (T, layer) in enumerate([(5, 0), (3, 1), (1, 2), (2, 3), (12, 4), (40, 5)]):
        ref, out = _run_pair(shape, T, layer)
        assert torch.isfinite(out.float()).all(), f"call {call}: output not written"
        diff = (out.float() - ref.float()).abs().max().item()
        rms = ref.float().square().mean().sqrt().item()
        assert diff <= 2e-2 * rms + 1e-3, f"call {call}: max |diff| {diff} vs rms {rms}"
        assert torch.equal(out, ref), f"call {call}: expected the identical kernel result"


def test_noalloc_reports_a_wait_that_ran_out_and_recovers():
    """A device-side wait that runs out during a call on the built-in array is readable through
    moe_sync_status(plan, NULL) before the next call, which starts from cleared status words again."""
    shape = wl.MoEShape("noalloc_to", 3, H=256, E=16, I=128, top_k=2, scoring=wl.SCORE_SOFTMAX)
    T = 2
    d = wl.make_layer(shape, T, device="cuda")
    plan = m.MoEPlan(shape.H, shape.E, shape.I, shape.top_k, shape.scoring, shape.renorm, T_max=T)
    plan.set_knob(0, "fused", 1)
    args = (d["hidden"], d["Wr"], d["bias"], d["W13q"], d["W13s"], d["W2q"], d["W2s"])
    ref = plan.forward(*args)
    plan.sync_status()
    assert m.load_library().moe_plan_set_timeout_ms(plan.handle, 5) == 0
    plan.set_knob(0, "debug_skip", 1)                            # the intermediate tile's readiness is never signalled
    out = torch.empty_like(ref)
    m.moe_forward_noalloc(plan.handle, T, *args, out)
    with pytest.raises(m.MoEError) as e:
        m.moe_sync_status(plan.handle, None)
    assert e.value.code == -7
    plan.set_knob(0, "debug_skip", 0)
    m.moe_forward_noalloc(plan.handle, T, *args, out)            # clears the array's status words itself
    m.moe_sync_status(plan.handle, None)
    assert torch.equal(out, ref)
    plan.close()


def test_noalloc_rejects_shapes_beyond_the_built_in_array():
    big = wl.SHAPES["c5_deepseek_v3"]                           # at T=64 this shape needs far more than 24 MiB
    h = m.moe_plan(big.H, big.E, big.I, big.top_k, big.scoring, big.renorm)
    x = torch.zeros(16, dtype=torch.uint8, device="cuda")
    with pytest.raises(m.MoEError) as e:
        m.moe_forward_noalloc(h, 64, x, x, x, x, x, x, x, x)
    assert e.value.code == -4 and "built-in array" in str(e.value)
    m.moe_plan_destroy(h)
