"""A device-side wait that runs out must end as an error status, never as a hang or a fault.

Every case starves one wait with "a flag that nothing sets" and a 5 ms limit, checks that the launch ends with
MOE_ERR_TIMEOUT, re-initialises the workspace and checks parity of the next step against the oracle:
  * the first grid-wide wait of either kernel variant (an arrival counter pre-loaded so that it never equals the grid
    size) -- nothing is in flight when the CTAs give up;
  * waits DEEPER in the pipeline, where the give-up has to wait for bulk copies in flight, let issued MMAs retire and
    free tensor memory before the CTA exits: the general variant's hand-over of the intermediate tile (its publish
    counters pre-loaded past their target), and the fused-unit variant's on-chip hand-over (the readiness signal left
    out through the plan's test hook).
"""
import pytest
import torch

from paper_2609_04244_b200 import MoEError, MoEPlan, load_library, moe_workspace_init, workloads as wl
from tests.parity import check_against_oracle

pytestmark = pytest.mark.gpu

SHAPE = wl.MoEShape("timeout_small", 9, H=256, E=16, I=128, top_k=2, scoring=wl.SCORE_SOFTMAX)
CTRL_WORDS = 64            # control words at the head of the workspace; the publish counters [2][8][E] follow
MAX_PASSES = 8


def _plan(T, fused):
    d = wl.make_layer(SHAPE, T, device="cuda")
    plan = MoEPlan(SHAPE.H, SHAPE.E, SHAPE.I, SHAPE.top_k, SHAPE.scoring, SHAPE.renorm, T_max=T)
    plan.set_knob(0, "fused", fused)
    assert plan.info(T)["fused"] == bool(fused)
    args = (d["hidden"], d["Wr"], d["bias"], d["W13q"], d["W13s"], d["W2q"], d["W2s"])
    assert load_library().moe_plan_set_timeout_ms(plan.handle, 5) == 0
    plan.forward(*args)
    plan.sync_status()                                   # a healthy launch first
    return d, plan, args


def _expect_timeout_then_recover(d, plan, args, T):
    plan.forward(*args)                                  # enqueues fine; the starved wait runs out on the device
    with pytest.raises(MoEError) as e:
        plan.sync_status()
    assert e.value.code == -7                            # MOE_ERR_TIMEOUT
    moe_workspace_init(plan.handle, plan.workspace)      # documented recovery
    dbg = plan.forward_debug(*args)
    plan.sync_status()
    r = check_against_oracle(SHAPE, T, d, dbg)
    assert r["rel_l2"] < 2e-3, r
    out2 = plan.forward(*args)                           # and the step after it is the same again
    plan.sync_status()
    assert torch.equal(out2, dbg["out"])


def test_wait_that_runs_out_returns_timeout_and_the_workspace_recovers():
    T = 3
    d, plan, args = _plan(T, fused=0)
    ctrl = plan.workspace[:4 * CTRL_WORDS].view(torch.int32)
    ctrl[3] = 1 << 20                                    # both routing arrival counters: can never equal the grid size
    ctrl[4] = 1 << 20
    torch.cuda.synchronize()
    _expect_timeout_then_recover(d, plan, args, T)
    plan.close()


def test_starved_handover_with_tiles_in_flight_general_variant():
    """The waits on an expert's publish counter (activation-tile producer, accumulator warps) run out while weight
    tiles are in flight and MMAs are issued: the teardown has to drain them."""
    T = 3
    d, plan, args = _plan(T, fused=0)
    words = plan.workspace[:4 * (CTRL_WORDS + 2 * MAX_PASSES * SHAPE.E)].view(torch.int32)
    torch.cuda.synchronize()
    par = (int(words[0].item()) + 1) & 1                 # the next launch counts in the counters of this parity
    lo = CTRL_WORDS + par * MAX_PASSES * SHAPE.E
    words[lo:lo + MAX_PASSES * SHAPE.E] = 1 << 20        # "published blocks" can never equal I/128 again
    torch.cuda.synchronize()
    _expect_timeout_then_recover(d, plan, args, T)
    plan.close()


def test_first_wait_of_the_fused_variant_runs_out():
    T = 2
    d, plan, args = _plan(T, fused=1)
    ctrl = plan.workspace[:4 * CTRL_WORDS].view(torch.int32)
    ctrl[8] = 1 << 20                                    # both "quantised input published" counters
    ctrl[9] = 1 << 20
    torch.cuda.synchronize()
    _expect_timeout_then_recover(d, plan, args, T)
    plan.close()


@pytest.mark.parametrize("cluster", [1, 2])
def test_starved_handover_with_tiles_in_flight_fused_variant(cluster):
    """The intermediate tile's readiness is never signalled (test hook): the MMA issuers, the accumulator warps, the
    producer and the final reduction all run out of time with tiles in flight; the next launch is healthy."""
    T = 2
    d, plan, args = _plan(T, fused=1)
    plan.set_knob(0, "cluster", cluster)
    plan.forward(*args)
    plan.sync_status()
    plan.set_knob(0, "debug_skip", 1)
    plan.forward(*args)
    with pytest.raises(MoEError) as e:
        plan.sync_status()
    assert e.value.code == -7
    plan.set_knob(0, "debug_skip", 0)
    moe_workspace_init(plan.handle, plan.workspace)
    dbg = plan.forward_debug(*args)
    plan.sync_status()
    r = check_against_oracle(SHAPE, T, d, dbg)
    assert r["rel_l2"] < 2e-3, r
    plan.close()
