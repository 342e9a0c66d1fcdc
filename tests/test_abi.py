"""The C-ABI library loads and exports every symbol the header declares (no compute without a GPU)."""
import ctypes
import os
import re

import pytest

import paper_2609_04244_b200 as m
from paper_2609_04244_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    src = open(os.path.join(ROOT, "include", "moe_b200.h")).read()
    src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
    return sorted(set(re.findall(r"\b(moe_[a-z_]+)\s*\(", src)))


def test_library_builds_and_exports_every_declared_symbol():
    path = build.build()
    lib = ctypes.CDLL(path)
    names = _declared()
    assert "moe_forward" in names and "moe_plan" in names and len(names) >= 10
    for n in names:
        assert hasattr(lib, n), n
    assert sorted(binding.EXPORTS) == [n for n in names if n in binding.EXPORTS]
    assert set(names) <= set(binding.EXPORTS) | {"moe_forward_noalloc"}


def test_no_cpu_fallback_without_device():
    import torch
    if torch.cuda.is_available():
        pytest.skip("has a GPU")
    with pytest.raises(m.MoEError) as e:
        m.moe_plan(2048, 128, 768, 8, 0, 1)
    assert e.value.code == -8


def test_plan_argument_validation_happens_before_any_device_work():
    lib = m.load_library()
    h = ctypes.c_void_p()
    assert lib.moe_plan(100, 8, 128, 2, 0, 1, ctypes.byref(h)) == -2          # H not a multiple of 128
    assert lib.moe_plan(128, 8, 128, 9, 0, 1, ctypes.byref(h)) == -2          # top_k > E
    assert lib.moe_plan(128, 8, 128, 2, 7, 1, ctypes.byref(h)) == -1          # unknown scoring
    assert lib.moe_plan(128, 8, 128, 2, 0, 1, None) == -1
    assert b"H and I" in lib.moe_last_error() or len(lib.moe_last_error()) > 0
    assert lib.moe_workspace_bytes(None, 4) == 0
    assert lib.moe_forward(None, 1, *([None] * 9), 0, None) == -1


def test_plan_helpers_reject_a_null_plan_without_touching_a_device():
    lib = binding.load_library()
    v = ctypes.c_int(-5)
    assert lib.moe_plan_set_knob(None, 0, 0, 4) == -1
    assert lib.moe_plan_get_knob(None, 0, 0, ctypes.byref(v)) == -1 and v.value == -5
    assert lib.moe_tokens_per_launch(None) == 0
    assert lib.moe_workspace_bytes(None, 8) == 0
    assert b"NULL" in lib.moe_last_error()
