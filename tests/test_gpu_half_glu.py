"""Half-GLU gate (ssm_glu_fwd / ssm_glu_bwd) against the oracle, through the C ABI: both
arithmetic paths (fp32 I/O on CUDA cores; bf16 I/O on the tensor-core GEMMs), ragged sizes,
repeated calls on one workspace, and the paper's block = SSM layer followed by the gate."""
import numpy as np
import pytest

from oracle import ssm_oracle as O
from paper_2502_20168_b200 import inputs as I
from tests.util import TOL, assert_close

pytestmark = pytest.mark.gpu


def _run(w):
    import torch
    from paper_2502_20168_b200 import binding as sb, harness
    d = I.draw_glu(w)
    io = torch.bfloat16 if w.io_dtype == "bf16" else torch.float32
    shape = sb.make_shape(w.B, w.T, w.H, 8, w.io_dtype)
    ws = sb.alloc_workspace(sb.ssm_glu_workspace_bytes(shape))
    W = harness.to_dev(d["W"])
    v, gout = harness.to_dev(d["v"], io), harness.to_dev(d["gout"], io)
    out, gv = torch.empty_like(v), torch.empty_like(v)
    dW = torch.empty_like(W)
    for _ in range(2):      # the workspace is reusable
        sb.ssm_glu_fwd(shape, W, v, out, ws)
        sb.ssm_glu_bwd(shape, W, v, gout, ws, gv, dW)
    sb.ssm_check(ws)
    tol = TOL[w.io_dtype]
    ref_out = O.half_glu_fwd(d["W"], d["v"])
    ref_gv, ref_dW = O.half_glu_bwd(d["W"], d["v"], d["gout"])
    errs = {"out": assert_close("out", harness.to_np(out), ref_out, tol),
            "gv": assert_close("gv", harness.to_np(gv), ref_gv, tol),
            "dW": assert_close("dW", harness.to_np(dW), ref_dW, tol)}
    print(w.name, {k: f"{e:.1e}" for k, e in errs.items()})


@pytest.mark.parametrize("B,T,H", [(1, 1, 8), (3, 17, 24), (2, 64, 256), (5, 33, 136)])
def test_gate_fp32(B, T, H):
    _run(I.Workload("glu32", B=B, T=T, H=H, P=8, io_dtype="f32", seed=B * 100 + T))


@pytest.mark.parametrize("B,T,H", [(3, 17, 24), (2, 100, 256), (4, 300, 128), (16, 1024, 512), (700, 66, 256)])
def test_gate_bf16(B, T, H):
    _run(I.Workload("glu16", B=B, T=T, H=H, P=8, io_dtype="bf16", seed=B * 100 + T))


def test_gate_at_the_sweep_size_bf16():
    _run(I.Workload("glu_c4", B=256, T=1024, H=512, P=8, io_dtype="bf16", seed=4))


def test_block_is_layer_then_gate():
    """y = SSM(u); out = half-GLU(y); backward through both, against the oracle's composition."""
    import torch
    from paper_2502_20168_b200 import binding as sb, harness
    w = I.Workload("block", B=4, T=40, H=32, P=16, io_dtype="f32", p_done=0.05, seed=31)
    d = I.draw_layer(w)
    g = I.draw_glu(w)
    buf = harness.LayerBuffers(d, "f32")
    buf.forward()
    shape = sb.make_shape(w.B, w.T, w.H, w.P, "f32")
    ws = sb.alloc_workspace(sb.ssm_glu_workspace_bytes(shape))
    W = harness.to_dev(g["W"])
    gout = harness.to_dev(g["gout"], torch.float32)
    out, gy = torch.empty_like(buf.y), torch.empty_like(buf.y)
    dW = torch.empty_like(W)
    sb.ssm_glu_fwd(shape, W, buf.y, out, ws)
    sb.ssm_glu_bwd(shape, W, buf.y, gout, ws, gy, dW)
    buf.gy = gy
    buf.backward()
    args = (d["Lambda"], d["Delta"], d["Bc"], d["Cc"], d["D"])
    y, _, _ = O.ssm_layer_fwd(*args, d["u"], d["done"], None)
    ref_out = O.half_glu_fwd(g["W"], y)
    ref_gy, ref_dW = O.half_glu_bwd(g["W"], y, g["gout"])
    ref = O.ssm_layer_bwd(*args, d["u"], d["done"], None, ref_gy)
    res = buf.results()
    assert_close("out", harness.to_np(out), ref_out, 1e-4)
    assert_close("dW", harness.to_np(dW), ref_dW, 1e-4)
    for k in ("du", "dLambda", "dDelta", "dB", "dC", "dD"):
        assert_close(k, res[k], ref[k], 1e-4)


def test_gate_argument_errors():
    import torch
    from paper_2502_20168_b200 import binding as sb
    shape = sb.make_shape(2, 3, 16, 8, "f32")
    ws = sb.alloc_workspace(sb.ssm_glu_workspace_bytes(shape))
    W = torch.zeros((16, 16), device="cuda")
    v = torch.zeros((2, 3, 16), device="cuda")
    with pytest.raises(sb.SsmError) as e:
        sb.ssm_glu_fwd(shape, W, v, None, ws)
    assert e.value.code == sb.SSM_ERR_NULL
    with pytest.raises(sb.SsmError) as e:
        sb.ssm_glu_fwd(shape, W, v, v.clone(), ws[:512])
    assert e.value.code == sb.SSM_ERR_WORKSPACE
