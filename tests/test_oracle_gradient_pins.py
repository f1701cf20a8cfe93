"""Pins for the oracle's hand-written backward pass: central finite differences on
every real and imaginary part, the adjoint (dot-product) identity, and an
independently derived gradient from autograd on a naive step-by-step loop."""
import numpy as np
import pytest
import torch

from oracle import ssm_oracle as O
from paper_2502_20168_b200 import inputs as I


def case(seed, B=2, T=6, H=3, P=4, p_done=0.3, x0=True):
    w = I.Workload("t", B=B, T=T, H=H, P=P, p_done=p_done, seed=seed)
    d = I.draw_layer(w, with_x0=x0, with_gxT=True)
    if d["done"] is not None:
        d["done"][0, 0] = 1          # flag on the first step with x0 given
        d["done"][-1, -1] = 1
    out = {k: (v.astype(np.complex128) if np.iscomplexobj(v) else v.astype(np.float64))
           for k, v in d.items() if isinstance(v, np.ndarray) and k != "done"}
    out["done"] = d["done"]
    if not x0:
        out["x0"] = None
    return out


def loss(d, **over):
    a = dict(d)
    a.update(over)
    y, xT, _ = O.ssm_layer_fwd(a["Lambda"], a["Delta"], a["Bc"], a["Cc"], a["D"], a["u"], a["done"], a["x0"])
    return float(np.sum(a["gy"] * y) + np.sum((np.conj(a["gxT"]) * xT).real))


def fd_grad(d, name, eps=1e-6):
    base = d[name]
    g = np.zeros(base.shape, np.complex128 if np.iscomplexobj(base) else np.float64)
    it = np.nditer(base, flags=["multi_index"])
    for _ in it:
        idx = it.multi_index
        for part in ((1.0, 1.0), (1j, 1j)) if np.iscomplexobj(base) else ((1.0, 1.0),):
            step, unit = part
            p = base.copy(); p[idx] += eps * step
            m = base.copy(); m[idx] -= eps * step
            g[idx] += unit * (loss(d, **{name: p}) - loss(d, **{name: m})) / (2 * eps)
    return g


@pytest.mark.parametrize("seed,p_done,x0", [(0, 0.0, False), (1, 0.3, True), (2, 0.5, True), (3, 0.3, False)])
def test_finite_differences_every_input(seed, p_done, x0):
    d = case(seed, p_done=p_done, x0=x0)
    g = O.ssm_layer_bwd(d["Lambda"], d["Delta"], d["Bc"], d["Cc"], d["D"], d["u"], d["done"],
                        d["x0"], d["gy"], d["gxT"])
    names = {"u": "du", "Lambda": "dLambda", "Delta": "dDelta", "Bc": "dB", "Cc": "dC", "D": "dD"}
    if x0:
        names["x0"] = "dx0"
    for inp, out in names.items():
        want = fd_grad(d, inp)
        scale = 1.0 + np.abs(want).max()
        assert np.abs(g[out] - want).max() < 2e-7 * scale, (inp, np.abs(g[out] - want).max())
    if x0 and d["done"] is not None:
        assert np.all(g["dx0"][0] == 0)          # first-step flag: x0 has no influence


def test_adjoint_identity_in_u_and_x0():
    d = case(5, B=3, T=9, H=4, P=5)
    rng = np.random.default_rng(0)
    du = rng.normal(size=d["u"].shape)
    dx0 = rng.normal(size=d["x0"].shape) + 1j * rng.normal(size=d["x0"].shape)
    args = (d["Lambda"], d["Delta"], d["Bc"], d["Cc"], d["D"])
    # the map (u, x0) -> (y, xT) is real-linear: J.delta = f(delta)
    jy, jxT, _ = O.ssm_layer_fwd(*args, du, d["done"], dx0)
    g = O.ssm_layer_bwd(*args, d["u"], d["done"], d["x0"], d["gy"], d["gxT"])
    lhs = np.sum(d["gy"] * jy) + np.sum((np.conj(d["gxT"]) * jxT).real)
    rhs = np.sum(g["du"] * du) + np.sum((np.conj(g["dx0"]) * dx0).real)
    assert abs(lhs - rhs) < 1e-11 * (1 + abs(lhs))


def test_scan_backward_alone_by_finite_differences():
    d = case(7, B=2, T=5, H=2, P=3)
    rng = np.random.default_rng(3)
    Abar = np.exp(d["Lambda"] * d["Delta"])
    Bu = rng.normal(size=(2, 5, 3)) + 1j * rng.normal(size=(2, 5, 3))
    gx = rng.normal(size=(2, 5, 3)) + 1j * rng.normal(size=(2, 5, 3))

    def f(Abar_, Bu_, x0_):
        x, xT = O.ssm_scan(Abar_, Bu_, d["done"], x0_)
        return float(np.sum((np.conj(gx) * x).real) + np.sum((np.conj(d["gxT"]) * xT).real))

    x, _ = O.ssm_scan(Abar, Bu, d["done"], d["x0"])
    gBu, gA, gx0 = O.ssm_scan_bwd(Abar, x, d["done"], d["x0"], gx, d["gxT"])
    eps = 1e-6
    for arr, got, pos in ((Abar, gA, 0), (Bu, gBu, 1), (d["x0"], gx0, 2)):
        it = np.nditer(arr, flags=["multi_index"])
        for _ in it:
            idx = it.multi_index
            want = 0j
            for step in (1.0, 1j):
                p = arr.copy(); p[idx] += eps * step
                m = arr.copy(); m[idx] -= eps * step
                a_p = [Abar, Bu, d["x0"]]; a_p[pos] = p
                a_m = [Abar, Bu, d["x0"]]; a_m[pos] = m
                want += step * (f(*a_p) - f(*a_m)) / (2 * eps)
            assert abs(got[idx] - want) < 1e-7 * (1 + abs(want))


def test_discretisation_backward_by_finite_differences_including_tiny_steps():
    rng = np.random.default_rng(1)
    lam = np.array([-0.01 + 0.002j, -0.5 + 3.0j, -1.0 + 0.1j])
    dt = np.array([1e-3, 0.1, 0.02])
    Bc = rng.normal(size=(3, 2)) + 1j * rng.normal(size=(3, 2))
    gA = rng.normal(size=3) + 1j * rng.normal(size=3)
    gB = rng.normal(size=(3, 2)) + 1j * rng.normal(size=(3, 2))

    def f(lam_, dt_, Bc_):
        A, Bb = O.zoh_discretize(lam_, dt_, Bc_)
        return float(np.sum((np.conj(gA) * A).real) + np.sum((np.conj(gB) * Bb).real))

    dL, dD, dB = O.zoh_discretize_bwd(lam, dt, Bc, gA, gB)
    for p in range(3):
        h = 1e-6 * abs(lam[p])
        want = 0j
        for step in (1.0, 1j):
            lp = lam.copy(); lp[p] += h * step
            lm = lam.copy(); lm[p] -= h * step
            want += step * (f(lp, dt, Bc) - f(lm, dt, Bc)) / (2 * h)
        assert abs(dL[p] - want) < 1e-6 * (1 + abs(want))
        h = 1e-6 * dt[p]
        tp = dt.copy(); tp[p] += h
        tm = dt.copy(); tm[p] -= h
        want = (f(lam, tp, Bc) - f(lam, tm, Bc)) / (2 * h)
        assert abs(dD[p] - want) < 1e-6 * (1 + abs(want))
    assert np.allclose(dB, np.conj((np.exp(lam * dt) - 1) / lam)[:, None] * gB, rtol=1e-9)


def test_autograd_on_a_naive_loop_agrees():
    """Independent derivation: torch autograd through the step-by-step definition."""
    d = case(9, B=2, T=7, H=3, P=4)
    t = {k: torch.tensor(v, requires_grad=True) for k, v in d.items()
         if k in ("Lambda", "Delta", "Bc", "Cc", "D", "u", "x0")}
    Abar = torch.exp(t["Lambda"] * t["Delta"])
    Bbar = ((Abar - 1) / t["Lambda"])[:, None] * t["Bc"]
    x = t["x0"]
    total = torch.zeros((), dtype=torch.float64)
    for k in range(7):
        keep = torch.tensor((d["done"][:, k] == 0).astype(np.float64))[:, None]
        x = Abar * (x * keep) + t["u"][:, k].to(torch.complex128) @ Bbar.T
        y = (x @ t["Cc"].T).real + t["D"] * t["u"][:, k]
        total = total + (torch.tensor(d["gy"][:, k]) * y).sum()
    total = total + (torch.conj(torch.tensor(d["gxT"])) * x).real.sum()
    total.backward()
    g = O.ssm_layer_bwd(d["Lambda"], d["Delta"], d["Bc"], d["Cc"], d["D"], d["u"], d["done"],
                        d["x0"], d["gy"], d["gxT"])
    pairs = {"u": "du", "Lambda": "dLambda", "Delta": "dDelta", "Bc": "dB", "Cc": "dC", "D": "dD", "x0": "dx0"}
    for inp, out in pairs.items():
        want = t[inp].grad.numpy()
        assert np.allclose(g[out], want, rtol=1e-9, atol=1e-11), inp


# ---- stacked model: GELU, LayerNorm, rounding points -------------------------
def test_gelu_and_layernorm_textbook_values():
    assert O.gelu(np.array([0.0]))[0] == 0.0
    assert abs(O.gelu(np.array([1.0]))[0] - 0.8413447460685429) < 1e-15      # Phi(1)
    assert abs(O.gelu(np.array([-1.0]))[0] + 0.15865525393145707) < 1e-15    # -Phi(-1)
    v = np.linspace(-4, 4, 41)
    fd = (O.gelu(v + 1e-6) - O.gelu(v - 1e-6)) / 2e-6
    assert np.allclose(O.gelu_grad(v), fd, atol=1e-8)
    z = np.random.default_rng(0).normal(size=(5, 16)) * 3 + 1
    out, zhat, rstd = O.layernorm_fwd(z, np.ones(16), np.zeros(16))
    assert np.allclose(out.mean(-1), 0, atol=1e-12) and np.allclose(out.var(-1), 1, atol=1e-4)
    want = torch.nn.functional.layer_norm(torch.tensor(z), (16,), eps=1e-5).numpy()
    assert np.allclose(out, want, atol=1e-12)


def _stack_case(seed=0, L=3, B=2, T=5, H=6, P=4):
    w = I.Workload("s", B=B, T=T, H=H, P=P, p_done=0.3, n_layers=L, seed=seed)
    d = I.draw_layer(w)
    rng = np.random.default_rng(seed + 100)
    params = [{k: (v.astype(np.complex128) if np.iscomplexobj(v) else v.astype(np.float64))
               for k, v in p.items()} for p in d["params"]]
    lnw = [1.0 + 0.1 * rng.normal(size=H) for _ in range(L)]
    lnb = [0.1 * rng.normal(size=H) for _ in range(L)]
    return params, lnw, lnb, d["u"].astype(np.float64), d["done"], d["gy"].astype(np.float64)


def test_stack_backward_by_finite_differences():
    params, lnw, lnb, u, done, gout = _stack_case()

    def f(params_=params, lnw_=lnw, lnb_=lnb, u_=u):
        out, _ = O.stack_fwd(params_, lnw_, lnb_, u_, done)
        return float(np.sum(gout * out))

    out, cache = O.stack_fwd(params, lnw, lnb, u, done)
    du, grads = O.stack_bwd(params, lnw, lnb, cache, done, gout)
    eps = 1e-6
    rng = np.random.default_rng(4)
    # input gradient: a sample of entries
    for _ in range(10):
        idx = tuple(rng.integers(0, s) for s in u.shape)
        up = u.copy(); up[idx] += eps
        um = u.copy(); um[idx] -= eps
        want = (f(u_=up) - f(u_=um)) / (2 * eps)
        assert abs(du[idx] - want) < 1e-6 * (1 + abs(want))
    # parameter gradients of the middle and bottom layers: a sample of entries each
    for l in (0, 1, 2):
        for name, gname in (("Lambda", "dLambda"), ("Delta", "dDelta"), ("Bc", "dB"), ("Cc", "dC"), ("D", "dD")):
            base = params[l][name]
            for _ in range(3):
                idx = tuple(rng.integers(0, s) for s in base.shape)
                want = 0j
                for step in ((1.0, 1j) if np.iscomplexobj(base) else (1.0,)):
                    pp = [dict(p) for p in params]; pm = [dict(p) for p in params]
                    a = base.copy(); a[idx] += eps * step; pp[l][name] = a
                    b = base.copy(); b[idx] -= eps * step; pm[l][name] = b
                    want += step * (f(params_=pp) - f(params_=pm)) / (2 * eps)
                got = grads[l][gname][idx]
                assert abs(got - want) < 2e-6 * (1 + abs(want)), (l, name)
        for arrs, gname, kw in ((lnw, "dln_weight", "lnw_"), (lnb, "dln_bias", "lnb_")):
            j = int(rng.integers(0, arrs[l].shape[0]))
            ap = [a.copy() for a in arrs]; ap[l][j] += eps
            am = [a.copy() for a in arrs]; am[l][j] -= eps
            want = (f(**{kw: ap}) - f(**{kw: am})) / (2 * eps)
            assert abs(grads[l][gname][j] - want) < 1e-6 * (1 + abs(want))


def test_stack_rounding_points_are_storage_values():
    params, lnw, lnb, u, done, gout = _stack_case(seed=1)
    u = I.round_to_bf16(u).astype(np.float64)
    out, cache = O.stack_fwd(params, lnw, lnb, u, done, round_io=I.round_to_bf16)
    assert np.array_equal(out, I.round_to_bf16(out))
    for c in cache:
        assert np.array_equal(c["v"], I.round_to_bf16(c["v"]))
        assert np.array_equal(c["u"], I.round_to_bf16(c["u"]))
    exact, _ = O.stack_fwd(params, lnw, lnb, u, done)
    assert np.abs(out - exact).max() < 0.05 and not np.array_equal(out, exact)
    du, _ = O.stack_bwd(params, lnw, lnb, cache, done, I.round_to_bf16(gout).astype(np.float64),
                        round_io=I.round_to_bf16)
    assert np.array_equal(du, I.round_to_bf16(du))
