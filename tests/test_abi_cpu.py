"""Host-side checks that need no GPU: the library loads, exports what the header declares,
and refuses bad arguments before touching a device."""
import ctypes
import os
import re

import pytest

from paper_2604_26294_b200 import binding as b
from paper_2604_26294_b200 import build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build_library()
    return b.load_library()


def _declared_functions():
    names = set()
    for header in ("tsp_mlp.h", "tsp_attn.h"):
        text = open(os.path.join(ROOT, "include", header)).read()
        text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
        names |= set(re.findall(r"\b(tsp_(?:mlp|attn)_\w+)\s*\(", text))
    return sorted(names)


def test_library_exports_every_declared_symbol(lib):
    names = _declared_functions()
    assert "tsp_mlp_plan" in names and "tsp_mlp_forward" in names and "tsp_mlp_backward" in names
    assert "tsp_attn_qkv_forward" in names and "tsp_attn_out_forward" in names and "tsp_mlp_ring_step" in names
    for n in names:
        assert hasattr(lib, n), f"{n} declared in include/ but not exported"
        assert n in b.SIGNATURES, f"{n} has no binding signature"
        assert callable(getattr(b, n)), f"binding lacks {n}"


def test_error_strings(lib):
    for code in range(-6, 1):
        assert b.error_string(code) not in ("", "unknown status")
    assert b.error_string(-99) == "unknown status"


def test_plan_rejects_bad_shapes_before_any_device_call(lib):
    out = ctypes.c_void_p()
    assert lib.tsp_mlp_plan(256, 768, 2, None) == b.TSP_ERR_INVALID_ARG
    assert lib.tsp_mlp_plan(0, 768, 2, ctypes.byref(out)) == b.TSP_ERR_INVALID_ARG
    assert lib.tsp_mlp_plan(256, 768, 0, ctypes.byref(out)) == b.TSP_ERR_INVALID_ARG
    assert lib.tsp_mlp_plan(256, 768, 65, ctypes.byref(out)) == b.TSP_ERR_INVALID_ARG
    assert lib.tsp_mlp_plan(256, 770, 4, ctypes.byref(out)) == b.TSP_ERR_UNSUPPORTED_SHAPE   # F % D
    assert lib.tsp_mlp_plan(256, 768, 4, ctypes.byref(out)) == b.TSP_ERR_UNSUPPORTED_SHAPE   # F/D = 192
    assert lib.tsp_mlp_plan(128, 768, 2, ctypes.byref(out)) == b.TSP_ERR_UNSUPPORTED_SHAPE   # H % 256
    assert not out.value


def test_null_plan_is_refused(lib):
    assert lib.tsp_mlp_forward(None, None, None, None, None, None, 256, 2, None) == b.TSP_ERR_INVALID_ARG
    assert lib.tsp_mlp_backward(None, *([None] * 9), 256, 2, None) == b.TSP_ERR_INVALID_ARG
    assert lib.tsp_mlp_workspace_bytes(None, 256, 0) == 0
    assert lib.tsp_mlp_status(None) == b.TSP_ERR_INVALID_ARG
    assert lib.tsp_mlp_plan_destroy(None) == b.TSP_ERR_INVALID_ARG


def test_no_gpu_means_loud_failure_not_fallback(lib):
    import torch

    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    with pytest.raises(b.TspError):
        b.tsp_mlp_plan(256, 768, 2)


def test_plan_options_defaults_and_validation(lib):
    o = b.tsp_mlp_options_default()
    assert o.struct_bytes == ctypes.sizeof(b.TspMlpOptions)
    assert all(getattr(o, n) == -1 for n, _ in b.TspMlpOptions._fields_[1:])
    out = ctypes.c_void_p()
    # option checks come before any device call, so they can be exercised without a GPU
    o.wide_mask = 8
    assert lib.tsp_mlp_plan_ex(256, 768, 2, ctypes.byref(o), ctypes.byref(out)) == b.TSP_ERR_INVALID_ARG
    o = b.tsp_mlp_options_default()
    o.struct_bytes = 8
    assert lib.tsp_mlp_plan_ex(256, 768, 2, ctypes.byref(o), ctypes.byref(out)) == b.TSP_ERR_INVALID_ARG
    o = b.tsp_mlp_options_default()
    o.timeout_ms = 0
    assert lib.tsp_mlp_plan_ex(256, 768, 2, ctypes.byref(o), ctypes.byref(out)) == b.TSP_ERR_INVALID_ARG
    o = b.tsp_mlp_options_default()
    o.rank_pair_tiles = 8
    assert lib.tsp_mlp_plan_ex(256, 768, 2, ctypes.byref(o), ctypes.byref(out)) == b.TSP_ERR_INVALID_ARG
    o = b.tsp_mlp_options_default()
    assert lib.tsp_mlp_plan_ex(128, 768, 2, ctypes.byref(o), ctypes.byref(out)) == b.TSP_ERR_UNSUPPORTED_SHAPE
    assert not out.value
    with pytest.raises(TypeError):
        b.tsp_mlp_plan_ex(256, 768, 2, no_such_field=1)
