"""Single-step mode (ssm_step_prepare / ssm_step) against the oracle's ssm_step, through the
C ABI: rollouts of several steps with the state handed from call to call (in place and out of
place), done flags, both arithmetic paths (fp32 I/O on CUDA cores, bf16 I/O on tensor cores at
an imagination-sized batch), and agreement with ssm_layer_fwd over the same steps."""
import numpy as np
import pytest

from oracle import ssm_oracle as O
from paper_2502_20168_b200 import inputs as I
from tests.util import TOL, assert_close

pytestmark = pytest.mark.gpu


def _rollout(w, steps, in_place):
    import torch
    from paper_2502_20168_b200 import binding as sb, harness
    d = I.draw_layer(I.small_variant(w, T=steps), with_x0=True)
    io = torch.bfloat16 if w.io_dtype == "bf16" else torch.float32
    shape = sb.make_shape(w.B, 1, w.H, w.P, w.io_dtype)
    dev = {k: harness.to_dev(d[k].astype(np.complex64)) for k in ("Lambda", "Bc", "Cc")}
    dev["Delta"] = harness.to_dev(d["Delta"].astype(np.float32))
    dev["D"] = harness.to_dev(d["D"].astype(np.float32))
    ws = sb.alloc_workspace(sb.ssm_step_workspace_bytes(shape))
    sb.ssm_step_prepare(shape, dev["Lambda"], dev["Delta"], dev["Bc"], dev["Cc"], ws)
    u = harness.to_dev(d["u"], io)                        # [B, steps, H]
    done = harness.to_dev(d["done"], torch.uint8) if d["done"] is not None else None
    x = harness.to_dev(d["x0"].astype(np.complex64))
    x_alt = torch.empty_like(x)
    y = torch.empty((w.B, w.H), dtype=io, device="cuda")
    ref_x = d["x0"]
    args = (d["Lambda"], d["Delta"], d["Bc"], d["Cc"], d["D"])
    tol = TOL[w.io_dtype]
    for t in range(steps):
        ut = u[:, t].contiguous()
        dt = None if done is None else done[:, t].contiguous()
        if in_place:
            sb.ssm_step(shape, dev["D"], ut, dt, x, x, y, ws)
        else:
            sb.ssm_step(shape, dev["D"], ut, dt, x, x_alt, y, ws)
            x, x_alt = x_alt, x
        sb.ssm_check(ws)
        ref_x, ref_y = O.ssm_step(*args, d["u"][:, t], None if d["done"] is None else d["done"][:, t], ref_x)
        assert_close(f"y step {t}", harness.to_np(y), ref_y, tol)
        assert_close(f"x step {t}", harness.to_np(x), ref_x, tol)
    return d, harness.to_np(x)


@pytest.mark.parametrize("in_place", [False, True])
def test_rollout_fp32_small_batch(in_place):
    _rollout(I.Workload("step32", B=16, T=1, H=256, P=128, io_dtype="f32", p_done=0.1, seed=21), 12, in_place)


def test_rollout_fp32_tiny_and_odd_sizes():
    _rollout(I.Workload("step_odd", B=3, T=1, H=40, P=24, io_dtype="f32", p_done=0.3, seed=22), 6, True)
    _rollout(I.Workload("step_p8", B=5, T=1, H=16, P=8, io_dtype="f32", p_done=0.0, seed=23), 4, False)


@pytest.mark.parametrize("in_place", [False, True])
def test_rollout_bf16_imagination_batch(in_place):
    # 32 x 128 start states, the paper's training batch, rolled out step by step
    _rollout(I.Workload("step_bf16", B=4096, T=1, H=512, P=256, io_dtype="bf16", p_done=0.01, seed=24), 5, in_place)


def test_steps_agree_with_the_parallel_form():
    """Context processed by ssm_layer_fwd, then stepping from its xT, equals one longer run."""
    import torch
    from paper_2502_20168_b200 import binding as sb, harness
    w = I.Workload("ctx", B=8, T=24, H=64, P=32, io_dtype="f32", p_done=0.05, seed=25)
    d = I.draw_layer(w)
    ctx = 16
    full = harness.run_layer(d, "f32")
    dc = dict(d, u=d["u"][:, :ctx], gy=d["gy"][:, :ctx], done=d["done"][:, :ctx])
    head = harness.run_layer(dc, "f32")
    assert_close("context y", head["y"], full["y"][:, :ctx], 1e-5)
    shape = sb.make_shape(w.B, 1, w.H, w.P, "f32")
    ws = sb.alloc_workspace(sb.ssm_step_workspace_bytes(shape))
    P = {k: harness.to_dev(d[k].astype(np.complex64)) for k in ("Lambda", "Bc", "Cc")}
    sb.ssm_step_prepare(shape, P["Lambda"], harness.to_dev(d["Delta"].astype(np.float32)), P["Bc"], P["Cc"], ws)
    D = harness.to_dev(d["D"].astype(np.float32))
    x = harness.to_dev(head["xT"].astype(np.complex64))
    y = torch.empty((w.B, w.H), dtype=torch.float32, device="cuda")
    for t in range(ctx, w.T):
        sb.ssm_step(shape, D, harness.to_dev(d["u"][:, t].astype(np.float32)),
                    harness.to_dev(d["done"][:, t], torch.uint8), x, x, y, ws)
        assert_close(f"y[{t}]", harness.to_np(y), full["y"][:, t], 1e-5)
    assert_close("final state", harness.to_np(x), full["xT"], 1e-5)


def test_step_argument_errors():
    import torch
    from paper_2502_20168_b200 import binding as sb
    shape = sb.make_shape(4, 1, 16, 8, "f32")
    ws = sb.alloc_workspace(sb.ssm_step_workspace_bytes(shape))
    D = torch.zeros(16, device="cuda")
    u = torch.zeros((4, 16), device="cuda")
    x = torch.zeros((4, 8), dtype=torch.complex64, device="cuda")
    y = torch.zeros((4, 16), device="cuda")
    with pytest.raises(sb.SsmError) as e:
        sb.ssm_step(shape, D, u, None, None, x, y, ws)
    assert e.value.code == sb.SSM_ERR_NULL
    with pytest.raises(sb.SsmError) as e:
        sb.ssm_step(shape, D, u, None, x, x, y, ws[:256])
    assert e.value.code == sb.SSM_ERR_WORKSPACE
