"""ssm_scan_bwd_static serves callers that may not allocate device memory when they call
the library (a plug-in inside a framework that owns the memory pool, a loop with a budget
fixed at start-up): it must give what ssm_scan_bwd gives with a caller workspace, and what
the float64 oracle gives, call after call, although every call reuses the same built-in
scratch array.

Collected last on purpose, so that a run that stops at the first failure has already run
every other test."""
import ctypes

import numpy as np
import pytest

from oracle import ssm_oracle as O

pytestmark = pytest.mark.gpu

TOL = 1e-4   # the fp32 tolerance of the other parity tests: max |a - b| <= TOL * (1 + |b|)


def _case(seed, B, T, P):
    import torch
    rng = np.random.default_rng(seed)
    lam = rng.uniform(-1.0, -0.01, P) + 1j * rng.uniform(0.0, np.pi, P)
    dt = np.exp(rng.uniform(np.log(1e-3), np.log(1e-1), P))
    c = lambda *s: (rng.normal(size=s) + 1j * rng.normal(size=s)).astype(np.complex64)
    dev = lambda a: torch.from_numpy(np.ascontiguousarray(a)).cuda()
    host = {"Abar": np.exp(lam * dt).astype(np.complex64), "done": (rng.random((B, T)) < 0.05).astype(np.uint8),
            "x0": c(B, P), "x": c(B, T, P), "gx": c(B, T, P), "gxT": c(B, P)}
    t = {k: dev(v) for k, v in host.items()}
    t["host"] = host
    return t


def _run(sb, shape, t, static):
    import torch
    B, T, P = shape.B, shape.T, shape.P
    out = {"gBu": torch.empty((B, T, P), dtype=torch.complex64, device="cuda"),
           "gAbar": torch.empty(P, dtype=torch.complex64, device="cuda"),
           "gx0": torch.empty((B, P), dtype=torch.complex64, device="cuda")}
    if static:
        sb.ssm_scan_bwd_static(shape, t["Abar"], t["done"], t["x0"], t["x"], t["gx"], t["gxT"],
                               out["gBu"], out["gAbar"], out["gx0"])
        sb.ssm_check_static()      # no bounded wait gave up (the status word lives in the static array)
    else:
        ws = sb.alloc_workspace(sb.ssm_scan_workspace_bytes(shape))
        sb.ssm_scan_bwd(shape, t["Abar"], t["done"], t["x0"], t["x"], t["gx"], t["gxT"],
                        out["gBu"], out["gAbar"], out["gx0"], ws)
        sb.ssm_check(ws)
    torch.cuda.synchronize()
    return {k: v.cpu().numpy() for k, v in out.items()}


def test_static_scratch_variant_matches_workspace_variant_on_two_calls_in_a_row():
    from paper_2502_20168_b200 import binding as sb
    # two different problems back to back: the second call finds the first one's leftovers
    cases = []
    for seed, (B, T, P) in enumerate([(6, 300, 64), (3, 129, 24)]):
        shape = sb.make_shape(B, T, 8, P, "f32")
        assert sb.ssm_scan_workspace_bytes(shape) <= sb.SSM_STATIC_SCRATCH_BYTES
        t = _case(seed, B, T, P)
        h = t["host"]
        s_ref, gA_ref, gx0_ref = O.ssm_scan_bwd(h["Abar"], h["x"], h["done"], h["x0"], h["gx"], h["gxT"])
        cases.append((shape, t, _run(sb, shape, t, static=False), {"gBu": s_ref, "gAbar": gA_ref, "gx0": gx0_ref}))
    for shape, t, want, ref in cases + cases[::-1]:        # static calls only, one after the other
        got = _run(sb, shape, t, static=True)
        for k in want:
            err = np.max(np.abs(got[k] - want[k]) / (1.0 + np.abs(want[k])))
            assert err <= TOL, (k, err)
            err = np.max(np.abs(got[k] - ref[k]) / (1.0 + np.abs(ref[k])))
            assert err <= TOL, ("against the oracle", k, err)


def test_static_scratch_variant_refuses_what_does_not_fit():
    from paper_2502_20168_b200 import binding as sb
    big = sb.make_shape(1 << 16, 4, 8, 512, "f32")
    assert sb.ssm_scan_workspace_bytes(big) > sb.SSM_STATIC_SCRATCH_BYTES
    ok = ctypes.c_void_p(4096)
    rc = sb.lib().ssm_scan_bwd_static(ctypes.byref(big), ok, None, None, ok, ok, None, ok, ok, None, None)
    assert rc == sb.SSM_ERR_TOO_LARGE
    assert "static buffer" in sb.status_string(rc)
