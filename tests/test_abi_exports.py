"""The shared library loads without a GPU and exports every symbol ssm.h declares;
host-side argument checks answer before anything is launched."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def sb():
    from paper_2502_20168_b200 import build
    build.build()
    from paper_2502_20168_b200 import binding
    return binding


def declared_functions():
    text = open(os.path.join(ROOT, "include", "ssm.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(ssm_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(sb):
    names = declared_functions()
    assert "ssm_layer_fwd" in names and "ssm_scan_bwd" in names and len(names) >= 10
    for n in names:
        assert hasattr(sb.lib(), n), n
    assert set(names) == set(sb.EXPORTS)


def test_status_strings(sb):
    assert sb.status_string(0) == "ok"
    seen = {sb.status_string(c) for c in range(-7, 1)}
    assert len(seen) == 8 and "unknown status" not in seen
    assert sb.status_string(-99) == "unknown status"


def test_host_side_argument_checks_need_no_gpu(sb):
    lib = sb.lib()
    good = sb.make_shape(2, 8, 16, 8, "f32")
    assert sb.ssm_layer_workspace_bytes(good) > 0 and sb.ssm_scan_workspace_bytes(good) > 0
    for bad in (sb.make_shape(0, 8, 16, 8, "f32"), sb.make_shape(2, 0, 16, 8, "f32"),
                sb.make_shape(2, 8, 12, 8, "f32"), sb.make_shape(2, 8, 16, 4, "f32")):
        assert sb.ssm_layer_workspace_bytes(bad) == 0
        assert lib.ssm_scan_fwd(ctypes.byref(bad), *([ctypes.c_void_p(256)] * 7), 1 << 20, None) == sb.SSM_ERR_SHAPE
    dt = sb.ssm_shape(2, 8, 16, 8, 5, 0)
    assert lib.ssm_discretize(ctypes.byref(dt), *([ctypes.c_void_p(256)] * 5), None) == sb.SSM_ERR_DTYPE
    null = ctypes.c_void_p(0)
    ok = ctypes.c_void_p(4096)
    assert lib.ssm_discretize(ctypes.byref(good), null, ok, ok, ok, ok, None) == sb.SSM_ERR_NULL
    assert lib.ssm_discretize(ctypes.byref(good), ctypes.c_void_p(4100), ok, ok, ok, ok, None) == sb.SSM_ERR_ALIGN
    assert lib.ssm_scan_fwd(ctypes.byref(good), ok, ok, null, null, ok, null, null, 0, None) == sb.SSM_ERR_WORKSPACE
    assert lib.ssm_scan_fwd(ctypes.byref(good), ok, ok, null, null, ok, null, ok, 16, None) == sb.SSM_ERR_WORKSPACE
    assert lib.ssm_scan_fwd(ctypes.byref(good), ok, ok, null, null, ok, null, ctypes.c_void_p(4112), 1 << 20, None) == sb.SSM_ERR_ALIGN
