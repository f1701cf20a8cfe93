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


def test_layer_plan_names_the_kernels_a_shape_takes(sb):
    """Host logic only (no GPU: the library then plans for 148 SMs, the B200's count): which projections and
    which form of the scans ssm_layer_fwd / ssm_layer_bwd take for the configurations of the benchmark."""
    plan = lambda *a: sb.ssm_layer_plan_string(sb.make_shape(*a))
    assert plan(1, 64, 32, 16, "f32") == "projections=cuda-cores scans=separate"              # H, P below a tile
    assert plan(16, 64, 256, 128, "f32") == "projections=tensor-cores-planes scans=separate"   # fp32 I/O
    fused = "projections=tensor-cores scans=fused chain_states=%d time_pairs=%d"
    assert plan(256, 1024, 512, 256, "bf16") == fused % (64, 0)     # the headline workload
    assert plan(4096, 64, 512, 256, "bf16") == fused % (64, 0)      # whole sequences inside a tile
    assert plan(32, 128, 512, 256, "bf16") == fused % (64, 0)       # the paper's batch: 64 chains
    assert plan(16, 128, 512, 256, "bf16") == fused % (32, 0)       # few sequences of one tile: narrow chains
    assert plan(16, 1024, 512, 256, "bf16") == fused % (64, 1)      # few long sequences: both CTAs on one
    assert plan(16, 16384, 512, 256, "bf16") == fused % (64, 1)
    assert plan(48, 1024, 512, 256, "bf16") == fused % (64, 1)      # 96 chains: three half-rounds beat two rounds
    assert plan(64, 4096, 512, 256, "bf16") == fused % (64, 0)      # 128 chains: four half-rounds do not
    assert plan(4, 1024, 512, 256, "bf16") == "projections=tensor-cores scans=separate"       # too few chains
    assert plan(3, 333, 512, 128, "bf16") == "projections=tensor-cores scans=separate"        # T not a multiple of 128
    # argument checks
    import ctypes
    buf = ctypes.create_string_buffer(8)
    assert sb.lib().ssm_layer_plan_string(ctypes.byref(sb.make_shape(2, 8, 16, 8, "f32")), None, 8) == sb.SSM_ERR_NULL
    assert sb.lib().ssm_layer_plan_string(ctypes.byref(sb.make_shape(2, 8, 12, 8, "f32")), buf, 8) == sb.SSM_ERR_SHAPE
    assert sb.lib().ssm_layer_plan_string(ctypes.byref(sb.make_shape(2, 8, 16, 8, "f32")), buf, 8) == sb.SSM_OK
    assert buf.value == b"project"   # cut to the buffer, terminated
