"""The offline schedule search (Section 3.4) on a small shape: it must emit a table, the table must apply, and the
tuned plan must still match the oracle."""
import json

import pytest

from paper_2609_04244_b200 import MoEPlan, workloads as wl
from paper_2609_04244_b200 import tune as tuner
from tests.parity import check_against_oracle

pytestmark = pytest.mark.gpu

SHAPE = wl.MoEShape("tune_small", 7, H=512, E=32, I=256, top_k=4, scoring=wl.SCORE_SOFTMAX)


def test_knobs_round_trip_and_reject_bad_values():
    plan = MoEPlan(SHAPE.H, SHAPE.E, SHAPE.I, SHAPE.top_k, SHAPE.scoring, SHAPE.renorm, T_max=16)
    assert plan.get_knob(8, "split_slack_kib") == 200 and plan.get_knob(8, "stages") == 0
    plan.set_knob(8, "split_slack_kib", 0)
    plan.set_knob(0, "stages", 6)
    assert plan.get_knob(8, "split_slack_kib") == 0 and plan.get_knob(4, "split_slack_kib") == 200
    assert plan.get_knob(16, "stages") == 6 and plan.info(8)["stages"] == 6
    with pytest.raises(Exception):
        plan.set_knob(8, "stages", 1)
    with pytest.raises(Exception):
        plan.set_knob(8, "compact_min", 40)
    assert plan.get_knob(16, "split_weight") == -1
    plan.set_knob(16, "split_weight", 8)
    assert plan.get_knob(16, "split_weight") == 8 and plan.get_knob(12, "split_weight") == -1
    with pytest.raises(Exception):
        plan.set_knob(16, "split_weight", 9)
    assert plan.get_knob(4, "fused") == -1 and plan.get_knob(4, "cluster") == 0
    plan.set_knob(4, "fused", 0)                          # the kernel variant is a per-token-count knob
    assert plan.get_knob(4, "fused") == 0 and plan.get_knob(3, "fused") == -1 and not plan.info(4)["fused"]
    plan.set_knob(4, "fused", 1)
    plan.set_knob(4, "cluster", 2)
    assert plan.info(4)["fused"] and plan.info(4)["cluster"] == 2
    with pytest.raises(Exception):
        plan.set_knob(4, "cluster", 3)
    plan.close()


def test_candidates_cover_both_kernel_variants_up_to_eight_tokens():
    small = tuner.candidates(4, 64, True)
    assert any(c["fused"] == 1 and c["cluster"] == 2 for c in small) and any(c["fused"] == 0 for c in small)
    assert all("fused" not in c for c in tuner.candidates(17, 64, True))
    assert all("fused" not in c for c in tuner.candidates(4, 64, False))


def test_search_emits_a_table_that_keeps_parity(tmp_path):
    table = tuner.tune(SHAPE, tokens=[1, 8], regimes=("natural", "same"), n_layers=2, steps=20, replays=1)
    assert set(table["per_tokens"]) == {"1", "8"} and table["plan"]["compact_min"] in (5, 9)
    for T in ("1", "8"):
        m = table["measured_us"][T]
        assert m["best"] > 0 and m["default"] > 0 and m["rejected"] == 0
    path = tmp_path / "schedule.json"
    path.write_text(json.dumps(table))
    schedule = json.loads(path.read_text())
    for T in (1, 8):
        d = wl.make_layer(SHAPE, T, device="cuda")
        plan = MoEPlan(SHAPE.H, SHAPE.E, SHAPE.I, SHAPE.top_k, SHAPE.scoring, SHAPE.renorm, T_max=8, schedule=schedule)
        for knob, value in schedule["per_tokens"][str(T)].items():
            assert plan.get_knob(T, knob) == value
        dbg = plan.forward_debug(d["hidden"], d["Wr"], d["bias"], d["W13q"], d["W13s"], d["W2q"], d["W2s"])
        plan.sync_status()
        r = check_against_oracle(SHAPE, T, d, dbg)
        assert r["rel_l2"] < 2e-3, r
        plan.close()
