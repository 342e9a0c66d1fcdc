"""Host logic of the offline schedule search that needs no GPU: which schedules are tried for a token count."""
from paper_2609_04244_b200 import tune as tuner


def test_both_kernel_variants_up_to_sixteen_tokens():
    small = tuner.candidates(4, 64, True)
    general = [c for c in small if c["fused"] == 0]
    fused = [c for c in small if c["fused"] == 1]
    assert general and fused
    assert {c["cluster"] for c in fused} == set(tuner.FUSED_CLUSTERS) and {c["stages"] for c in fused} == set(tuner.FUSED_STAGES)
    assert all(c["cluster"] == 0 for c in general)
    # the general variant's own knob grid is complete
    n = 1
    for values in tuner.relevant_knobs(4, 64).values():
        n *= len(values)
    assert len(general) == n


def test_no_variant_choice_beyond_sixteen_tokens_or_where_the_shape_does_not_admit_it():
    assert all("fused" not in c for c in tuner.candidates(17, 64, True))
    assert all("fused" not in c for c in tuner.candidates(4, 64, False))
    assert all("fused" in c for c in tuner.candidates(16, 64, True))


def test_defaults_are_the_first_value_of_every_grid():
    for knob, values in tuner.PER_TOKEN_GRID.items():
        assert tuner.plan_default(knob, 1) == values[0] or knob == "split_slack_kib"
    assert tuner.plan_default("split_slack_kib", 8) == 200 and tuner.plan_default("split_slack_kib", 9) == 100
    assert tuner.plan_default("fused") == -1 and tuner.plan_default("cluster") == 0


def test_route_all_and_split_weight_only_where_they_matter():
    assert tuner.relevant_knobs(4, 64)["route_all_tokens"] == [8] and tuner.relevant_knobs(4, 64)["split_weight"] == [-1]
    assert len(tuner.relevant_knobs(16, 64)["route_all_tokens"]) > 1 and len(tuner.relevant_knobs(16, 64)["split_weight"]) > 1
    assert tuner.relevant_knobs(64, 64)["route_all_tokens"] == [8]
