"""Host-side checks of the input generators and the roofline byte counts.  CPU only."""
import os

import numpy as np
import torch

import oracle
from paper_2609_04244_b200 import workloads as wl

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def test_paper_closed_forms_golden():
    for line in open(os.path.join(GOLD, "paper_closed_forms.txt")):
        if line.startswith("#") or not line.strip():
            continue
        key, *v = line.split()
        if key == "k_over_E":
            assert int(v[0]) / int(v[1]) == float(v[2])
        elif key == "padded_fraction_rows":
            assert 1 - int(v[0]) / int(v[1]) == float(v[2])
        elif key == "U":
            assert wl.expected_unique_experts(int(v[0]), int(v[1]), int(v[2])) == float(v[3])
    assert abs(wl.expected_unique_experts(128, 8, 8) - 51.6) < 0.1


def test_algorithmic_bytes_match_eq5_plus_extras():
    s = wl.SHAPES["c2_qwen3_30b_a3b"]
    assert s.bytes_per_expert == 3 * 2048 * 768 + 4 * (12 * 16 + 16 * 6)
    assert wl.algorithmic_bytes(s, 1, 8) == 8 * s.bytes_per_expert + 2 * 128 * 2048 + 4 * 2048
    s5 = wl.SHAPES["c5_deepseek_v3"]
    assert wl.algorithmic_bytes(s5, 1, 8) == 8 * (3 * 7168 * 2048 + 4 * (32 * 56 + 56 * 16)) + 2 * 256 * 7168 + 4 * 256 + 4 * 7168


def test_seeds_distinct_and_generation_reproducible():
    s = wl.SHAPES["c1_tiny"]
    seeds = {wl.workload_seed(s, T, r, l) for T in (1, 2, 64) for r in wl.REGIMES for l in (0, 1)}
    assert len(seeds) == 18
    a = wl.make_layer(s, 2, experts=[0, 3])
    b = wl.make_layer(s, 2, experts=[3])
    assert torch.equal(a["W13q"][3], b["W13q"][3]) and torch.equal(a["W2s"][3], b["W2s"][3])
    assert torch.equal(a["hidden"], b["hidden"]) and torch.equal(a["Wr"], b["Wr"])
    assert not b["W13q"][0].any()


def test_block_packing_statistics_and_dequant_error():
    g = torch.Generator().manual_seed(0)
    m = torch.randn(256, 384, generator=g) * 0.02
    q, s = wl.pack_fp8_blockwise(m)
    assert q.dtype == torch.uint8 and s.shape == (2, 3)
    deq = q.view(torch.float8_e4m3fn).float() * s.repeat_interleave(128, 0).repeat_interleave(128, 1)
    assert ((deq - m).abs() <= m.abs() * 2 ** -4 + s.max() * 2 ** -10).all()
    assert (q.view(-1) & 0x7F).max() == 0x7E       # every block's amax maps to 448


def test_forced_routing_regimes_realise_intended_experts():
    s = wl.MoEShape("t", 3, H=512, E=32, I=128, top_k=4, scoring=wl.SCORE_SOFTMAX)
    for T in (1, 4, 8):
        for regime, want_u in (("same", 4), ("disjoint", min(32, 4 * T))):
            d = wl.make_layer(s, T, regime=regime)
            r = oracle.moe_forward(d["hidden"].view(torch.int16).numpy().view(np.uint16),
                                   d["Wr"].view(torch.int16).numpy().view(np.uint16), None,
                                   d["W13q"].numpy(), d["W13s"].numpy(), d["W2q"].numpy(), d["W2s"].numpy(),
                                   top_k=4)
            assert len(np.unique(r["ids"])) == want_u, (T, regime)
            if regime == "same":
                assert (np.sort(r["ids"], axis=1) == np.arange(4)).all()
            else:
                for t in range(T):
                    assert sorted(r["ids"][t]) == sorted((4 * t + j) % 32 for j in range(4))
