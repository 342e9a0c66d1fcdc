"""Pins for the oracle's scalar codecs and group quantiser (CPU only).

Sources that fix the expected values: the E4M3 format definition (closed form),
torch's own float8_e4m3fn / bfloat16 casts (library routines written by someone
else), exhaustively enumerated rounding midpoints, and hand-worked groups in
tests/golden/.
"""
import math
import os

import numpy as np
import pytest
import torch

import oracle

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _closed_form(code):
    s, e, m = code >> 7, (code >> 3) & 15, code & 7
    if e == 15 and m == 7:
        return math.nan
    v = (m / 8.0) * 2.0 ** -6 if e == 0 else (1 + m / 8.0) * 2.0 ** (e - 7)
    return -v if s else v


def test_e4m3_decode_all_codes_closed_form_and_torch():
    lut = torch.arange(256, dtype=torch.uint8).view(torch.float8_e4m3fn).to(torch.float32).numpy()
    for c in range(256):
        got = oracle.e4m3_to_double(c)
        want = _closed_form(c)
        if math.isnan(want):
            assert math.isnan(got) and math.isnan(lut[c])
        else:
            assert got == want == float(lut[c])
            assert math.copysign(1.0, got) == math.copysign(1.0, want)


def test_e4m3_spot_codes_golden():
    for line in open(os.path.join(GOLD, "e4m3_spot_codes.txt")):
        if line.startswith("#") or not line.strip():
            continue
        code, val = line.split()
        got = oracle.e4m3_to_double(int(code, 16))
        assert got == float(val) and math.copysign(1, got) == math.copysign(1, float(val))
    assert math.isnan(oracle.e4m3_to_double(0x7F)) and math.isnan(oracle.e4m3_to_double(0xFF))


def test_e4m3_encode_roundtrip_identity():
    for c in range(256):
        v = _closed_form(c)
        if math.isnan(v):
            continue
        assert oracle.e4m3_from_float(v) == c


def test_e4m3_encode_midpoints_tie_to_even_and_neighbours():
    pos = sorted(_closed_form(c) for c in range(0x7F))  # all non-negative finite values, ascending == code order
    for c in range(0x7E):
        lo, hi = pos[c], pos[c + 1]
        mid = (lo + hi) / 2.0                      # exactly representable in fp32
        even = c if (c & 1) == 0 else c + 1
        assert oracle.e4m3_from_float(mid) == even, (c, mid)
        assert oracle.e4m3_from_float(-mid) == (even | 0x80)
        below = np.nextafter(np.float32(mid), np.float32(0))
        above = np.nextafter(np.float32(mid), np.float32(1e9))
        assert oracle.e4m3_from_float(below) == c
        assert oracle.e4m3_from_float(above) == c + 1


def test_e4m3_encode_saturation_nan_signed_zero():
    for v in (448.0, 449.0, 464.0, 465.0, 480.0, 1e9, math.inf):
        assert oracle.e4m3_from_float(v) == 0x7E
        assert oracle.e4m3_from_float(-v) == 0xFE
    assert oracle.e4m3_from_float(math.nan) & 0x7F == 0x7F
    assert oracle.e4m3_from_float(0.0) == 0x00
    assert oracle.e4m3_from_float(-0.0) == 0x80
    assert oracle.e4m3_from_float(-1e-12) == 0x80
    assert oracle.e4m3_from_float(2.0 ** -10) == 0x00      # tie between 0 and 2^-9 -> even (0)
    assert oracle.e4m3_from_float(3 * 2.0 ** -10) == 0x02  # tie between 1 and 2 subnormal steps -> 2


def test_e4m3_encode_matches_torch_cast_on_random_values():
    rng = np.random.default_rng(1)
    x = np.concatenate([rng.standard_normal(20000) * s for s in (1e-3, 0.05, 1.0, 30.0, 300.0)]).astype(np.float32)
    want = torch.from_numpy(x).clamp(-448, 448).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    got = np.array([oracle.e4m3_from_float(v) for v in x], dtype=np.uint8)
    assert np.array_equal(got, want)


def test_bf16_codec_matches_torch_and_rounds_once():
    bits = np.arange(0, 65536, 7, dtype=np.uint32).astype(np.uint16)
    ref = torch.from_numpy(bits.view(np.int16)).view(torch.bfloat16).to(torch.float64).numpy()
    for b, r in zip(bits[:3000], ref[:3000]):
        got = oracle.bf16_to_double(int(b))
        assert (math.isnan(got) and math.isnan(r)) or got == r
    rng = np.random.default_rng(2)
    x = (rng.standard_normal(20000) * np.exp(rng.uniform(-20, 20, 20000))).astype(np.float32)
    want = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    got = np.array([oracle.double_to_bf16(float(v)) for v in x], dtype=np.uint16)
    assert np.array_equal(got, want)
    # a double that double-rounding through fp32 would get wrong: 1 + 2^-8 + 2^-30 must round UP to 1 + 2^-7
    assert oracle.double_to_bf16(1.0 + 2.0 ** -8 + 2.0 ** -30) == 0x3F81
    assert oracle.double_to_bf16(1.0 + 2.0 ** -8) == 0x3F80          # exact tie -> even
    assert oracle.double_to_bf16(1.0 + 3 * 2.0 ** -8) == 0x3F82      # tie -> even (up)
    assert oracle.double_to_bf16(1.4621171572600098) == 0x3FBB
    assert oracle.double_to_bf16(-0.0) == 0x8000
    assert oracle.double_to_bf16(2.0 ** -133) == 0x0001 and oracle.double_to_bf16(2.0 ** -134) == 0x0000


def _golden_groups():
    g = {}
    for line in open(os.path.join(GOLD, "quant_worked_groups.txt")):
        if line.startswith("#") or not line.strip():
            continue
        name, key, *vals = line.split()
        g.setdefault(name, {})[key] = vals
    return g


@pytest.mark.parametrize("name", ["A", "B"])
def test_quantize_worked_groups_golden(name):
    g = _golden_groups()[name]
    x = np.zeros(128, np.float32)
    vals = [float(v) for v in g["x"]]
    x[: len(vals)] = vals
    q, s = oracle.quantize_groups(x, 128)
    assert s[0] == np.float32(float(g["scale"][0]))
    assert [int(b, 16) for b in g["bytes"]] == list(q[: len(vals)])
    assert all(b == 0 for b in q[len(vals):])


def test_quantize_groups_matches_torch_pipeline_and_zero_group():
    rng = np.random.default_rng(3)
    x = torch.from_numpy(rng.standard_normal(128 * 64).astype(np.float32)).to(torch.bfloat16).to(torch.float32)
    x[128:256] = 0.0
    x[300] = -0.0
    q, s = oracle.quantize_groups(x.numpy(), 128)
    v = x.view(-1, 128)
    sc = (v.abs().amax(dim=1).clamp_min(1e-10) / 448.0)
    want = (v / sc[:, None]).clamp(-448, 448).to(torch.float8_e4m3fn).view(torch.uint8).numpy().ravel()
    assert np.array_equal(s, sc.numpy())
    assert np.array_equal(q, want)
    assert s[1] == np.float32(1e-10) / np.float32(448.0) and not q[128:256].any()
    # power-of-two input scaling: same bytes, scale multiplied exactly
    q2, s2 = oracle.quantize_groups((x * 8.0).numpy(), 128)
    keep = np.arange(64) != 1
    assert np.array_equal(q2, q) and np.array_equal(s2[keep], s[keep] * 8)
