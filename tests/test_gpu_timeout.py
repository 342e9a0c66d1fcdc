"""A device-side wait that runs out must end as an error status, never as a hang: the first grid-wide wait of the kernel
is made to run out (its arrival counter is pre-loaded so that it can never reach the grid size) with a 5 ms limit."""
import pytest
import torch

from paper_2609_04244_b200 import MoEError, MoEPlan, load_library, moe_workspace_init, workloads as wl
from tests.parity import check_against_oracle

pytestmark = pytest.mark.gpu

SHAPE = wl.MoEShape("timeout_small", 9, H=256, E=16, I=128, top_k=2, scoring=wl.SCORE_SOFTMAX)


def test_wait_that_runs_out_returns_timeout_and_the_workspace_recovers():
    T = 3
    d = wl.make_layer(SHAPE, T, device="cuda")
    plan = MoEPlan(SHAPE.H, SHAPE.E, SHAPE.I, SHAPE.top_k, SHAPE.scoring, SHAPE.renorm, T_max=T)
    args = (d["hidden"], d["Wr"], d["bias"], d["W13q"], d["W13s"], d["W2q"], d["W2s"])
    assert load_library().moe_plan_set_timeout_ms(plan.handle, 5) == 0
    plan.forward(*args)
    plan.sync_status()                                   # a healthy launch first
    ctrl = plan.workspace[:256].view(torch.int32)
    ctrl[3] = 1 << 20                                    # both routing arrival counters: can never equal the grid size
    ctrl[4] = 1 << 20
    torch.cuda.synchronize()
    plan.forward(*args)                                  # enqueues fine; every CTA gives up at its first grid-wide wait
    with pytest.raises(MoEError) as e:
        plan.sync_status()
    assert e.value.code == -7                            # MOE_ERR_TIMEOUT
    moe_workspace_init(plan.handle, plan.workspace)      # documented recovery
    dbg = plan.forward_debug(*args)
    plan.sync_status()
    r = check_against_oracle(SHAPE, T, d, dbg)
    assert r["rel_l2"] < 2e-3, r
    plan.close()
