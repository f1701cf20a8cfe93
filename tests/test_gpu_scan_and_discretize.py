"""Stand-alone entry points (ssm_discretize, ssm_discretize_bwd, ssm_scan_fwd, ssm_scan_bwd)
against the oracle, through the C ABI: both scan kernels (streaming tiles of several group
widths; one thread per sequence for fewer than 16 states), in place and out of place, ragged
last tiles, error paths."""
import numpy as np
import pytest

from oracle import ssm_oracle as O
from tests.util import assert_close

pytestmark = pytest.mark.gpu

TOL = 1e-4


def _dev(a):
    import torch
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def _c(rng, *s):
    return (rng.normal(size=s) + 1j * rng.normal(size=s)).astype(np.complex64)


def _abar(rng, P):
    lam = rng.uniform(-1.0, -0.01, P) + 1j * rng.uniform(0.0, np.pi, P)
    dt = np.exp(rng.uniform(np.log(1e-3), np.log(1e-1), P))
    return np.exp(lam * dt).astype(np.complex64)


# (B, T, P): P = 8 or T < 8 -> one thread per sequence; otherwise tiles of 16..128 states, the narrow ones
# when B is small; T around multiples of the tile heights; P that is not a multiple of the width
SCAN_SHAPES = [(1, 1, 8), (2, 63, 8), (3, 64, 24), (2, 65, 40), (1, 1000, 264), (4, 517, 128),
               (2, 4100, 16), (800, 70, 256), (40, 129, 136), (600, 33, 128), (5, 256, 64), (300, 1, 128),
               (7, 7, 32), (6, 8, 32),
               # few sequences, long: narrow chains, many tiles per chain (ragged ends, P off the width)
               (2, 5000, 128), (3, 1100, 64), (16, 1200, 256), (9, 2100, 136), (1, 1024, 64), (4, 1025, 192)]


@pytest.mark.parametrize("B,T,P", SCAN_SHAPES)
@pytest.mark.parametrize("flags", ["none", "sparse", "dense"])
def test_scan_fwd_and_bwd(B, T, P, flags):
    import torch
    from paper_2502_20168_b200 import binding as sb
    rng = np.random.default_rng(B * 7919 + T * 31 + P)
    A = _abar(rng, P)
    Bu, gx = _c(rng, B, T, P), _c(rng, B, T, P)
    x0, gxT = _c(rng, B, P), _c(rng, B, P)
    done = None
    if flags != "none":
        done = (rng.random((B, T)) < (0.004 if flags == "sparse" else 0.3)).astype(np.uint8)
        done[0, 0] = 1
        done[-1, -1] = 1
    shape = sb.make_shape(B, T, 8, P, "f32")
    ws = sb.alloc_workspace(sb.ssm_scan_workspace_bytes(shape))
    dA, dBu, dx0, dgx, dgxT = _dev(A), _dev(Bu), _dev(x0), _dev(gx), _dev(gxT)
    ddone = None if done is None else _dev(done)
    x = torch.empty_like(dBu)
    xT = torch.empty_like(dx0)
    sb.ssm_scan_fwd(shape, dA, dBu, ddone, dx0, x, xT, ws)
    sb.ssm_check(ws)
    ref_x, ref_xT = O.ssm_scan(A, Bu, done, x0)
    assert_close("x", x.cpu().numpy(), ref_x, TOL)
    assert_close("xT", xT.cpu().numpy(), ref_xT, TOL)
    # in place, no x0, no xT
    buf = dBu.clone()
    sb.ssm_scan_fwd(shape, dA, buf, ddone, None, buf, None, ws)
    assert_close("x in place", buf.cpu().numpy(), O.ssm_scan(A, Bu, done, None)[0], TOL)

    gBu = torch.empty_like(dgx)
    gA = torch.empty(P, dtype=torch.complex64, device="cuda")
    gx0 = torch.empty_like(dx0)
    sb.ssm_scan_bwd(shape, dA, ddone, dx0, x, dgx, dgxT, gBu, gA, gx0, ws)
    sb.ssm_check(ws)
    r_s, r_gA, r_gx0 = O.ssm_scan_bwd(A, x.cpu().numpy(), done, x0, gx, gxT)
    assert_close("gBu", gBu.cpu().numpy(), r_s, TOL)
    assert_close("gx0", gx0.cpu().numpy(), r_gx0, TOL)
    assert_close("gAbar", gA.cpu().numpy(), r_gA, TOL)
    # in place over gx, without gxT / x0 / gx0
    buf = dgx.clone()
    sb.ssm_scan_bwd(shape, dA, ddone, None, x, buf, None, buf, gA, None, ws)
    r_s2, _, _ = O.ssm_scan_bwd(A, x.cpu().numpy(), done, None, gx, None)
    assert_close("gBu in place", buf.cpu().numpy(), r_s2, TOL)


@pytest.mark.parametrize("H,P", [(8, 8), (40, 24), (512, 256)])
def test_discretize_and_its_adjoint(H, P):
    import torch
    from paper_2502_20168_b200 import binding as sb
    rng = np.random.default_rng(H + P)
    lam = (rng.uniform(-1.0, -0.01, P) + 1j * rng.uniform(0.0, np.pi, P)).astype(np.complex64)
    lam[0] = -0.01 + 1e-4j            # tiny |Lambda Delta|: exp(z) - 1 must not cancel
    dt = np.exp(rng.uniform(np.log(1e-3), np.log(1e-1), P)).astype(np.float32)
    dt[0] = 1e-3
    Bc = _c(rng, P, H)
    gA, gB = _c(rng, P), _c(rng, P, H)
    shape = sb.make_shape(1, 1, H, P, "f32")
    Abar = torch.empty(P, dtype=torch.complex64, device="cuda")
    Bbar = torch.empty((P, H), dtype=torch.complex64, device="cuda")
    sb.ssm_discretize(shape, _dev(lam), _dev(dt), _dev(Bc), Abar, Bbar)
    rA, rB = O.zoh_discretize(lam, dt, Bc)
    assert np.abs(Abar.cpu().numpy() - rA).max() < 2e-7
    assert np.max(np.abs(Bbar.cpu().numpy() - rB) / np.abs(rB)) < 1e-6      # relative: no cancellation
    dL = torch.empty(P, dtype=torch.complex64, device="cuda")
    dD = torch.empty(P, dtype=torch.float32, device="cuda")
    dB = torch.empty((P, H), dtype=torch.complex64, device="cuda")
    sb.ssm_discretize_bwd(shape, _dev(lam), _dev(dt), _dev(Bc), _dev(gA), _dev(gB), dL, dD, dB)
    rL, rD, rdB = O.zoh_discretize_bwd(lam, dt, Bc, gA, gB)
    assert_close("dLambda", dL.cpu().numpy(), rL, TOL)
    assert_close("dDelta", dD.cpu().numpy(), rD, TOL)
    assert_close("dB", dB.cpu().numpy(), rdB, TOL)


def test_calls_are_refused_cleanly_and_leave_the_context_usable():
    import torch
    from paper_2502_20168_b200 import binding as sb
    shape = sb.make_shape(2, 8, 8, 8, "f32")
    t = torch.zeros(2 * 8 * 8, dtype=torch.complex64, device="cuda")
    small_ws = torch.empty(256, dtype=torch.uint8, device="cuda")
    with pytest.raises(sb.SsmError) as e:
        sb.ssm_scan_fwd(shape, t, t, None, None, t, None, small_ws)
    assert e.value.code == sb.SSM_ERR_WORKSPACE
    with pytest.raises(sb.SsmError) as e:
        sb.ssm_scan_fwd(shape, t, None, None, None, t, None, small_ws)
    assert e.value.code == sb.SSM_ERR_NULL
    ws = sb.alloc_workspace(sb.ssm_scan_workspace_bytes(shape))
    off = t.view(torch.float32)[1:]                      # 4-byte offset: misaligned
    with pytest.raises(sb.SsmError) as e:
        sb.ssm_scan_fwd(shape, t, off, None, None, t, None, ws)
    assert e.value.code == sb.SSM_ERR_ALIGN
    sb.ssm_scan_fwd(shape, t, t, None, None, t, None, ws)   # still works afterwards
    sb.ssm_check(ws)
    torch.cuda.synchronize()
