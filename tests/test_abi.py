"""The C-ABI library loads and exports every function that include/moe.h declares.
No compute call is made here (there may be no GPU)."""
import ctypes
import os
import re

import pytest
import torch

from paper_2509_02753_b200 import binding as B

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "moe.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(moe_[a-z0-9_]+)\s*\(", text)))


def test_library_exports_every_declared_entry_point():
    lib = B.load_library()
    names = _declared()
    assert "moe_layer_forward" in names and "moe_stack_forward" in names and "moe_plan_create" in names
    for n in names:
        assert hasattr(lib, n), f"{n} declared in moe.h but not exported"
    assert set(names) == set(B.EXPORTS)


def test_status_strings():
    assert B.status_string(0) == "ok"
    for code in range(-8, 0):
        assert B.status_string(code) not in ("ok", "unknown status")
    assert B.status_string(-99) == "unknown status"


def test_struct_layouts_match_the_header():
    assert ctypes.sizeof(B.moe_config_t) == 9 * 4
    assert ctypes.sizeof(B.moe_layer_weights_t) == 9 * ctypes.sizeof(ctypes.c_void_p)


def test_plan_create_rejects_bad_configs_before_touching_the_device():
    lib = B.load_library()
    out = ctypes.c_void_p()
    assert lib.moe_plan_create(None, ctypes.byref(out)) == -1
    cfg = B.moe_config_t(256, 8, 512, 0, 0, 8, 9, B.MOE_BF16, 1.0)      # max_k > E
    assert lib.moe_plan_create(ctypes.byref(cfg), ctypes.byref(out)) == -1
    cfg = B.moe_config_t(250, 8, 512, 0, 0, 8, 2, B.MOE_BF16, 1.0)      # d % 8
    assert lib.moe_plan_create(ctypes.byref(cfg), ctypes.byref(out)) == -2
    cfg = B.moe_config_t(256, 200, 512, 0, 0, 8, 2, B.MOE_BF16, 1.0)    # E too large
    assert lib.moe_plan_create(ctypes.byref(cfg), ctypes.byref(out)) == -2
    assert out.value is None


@pytest.mark.skipif(torch.cuda.is_available(), reason="checks the no-device path")
def test_no_device_means_an_error_not_a_fallback():
    with pytest.raises(B.MoEError) as e:
        B.MoEPlan(256, 8, 512, 8, 2, torch.bfloat16)
    assert e.value.status == -5
