"""Pins for the float64 oracle's forward path: each test fixes it to something the
paper or the mathematics determines, not to a second copy of its own formula."""
import math
import random

import numpy as np
import pytest
from scipy.integrate import solve_ivp
from scipy.signal import lfilter

from oracle import ssm_oracle as O
from paper_2502_20168_b200 import inputs as I


def small(seed=0, B=2, T=7, H=3, P=4, p_done=0.0, **kw):
    w = I.Workload("t", B=B, T=T, H=H, P=P, p_done=p_done, seed=seed)
    return I.draw_layer(w, **kw)


def bracket_fold(elems, op, rng):
    """Combine a list with a random (but order-preserving) bracketing."""
    elems = list(elems)
    while len(elems) > 1:
        i = rng.randrange(len(elems) - 1)
        elems[i:i + 2] = [op(elems[i], elems[i + 1])]
    return elems[0]


# ---- discretisation -------------------------------------------------------
def test_zoh_matches_integrating_the_ode():
    """ZOH is exact sampling of dx/dt = Lambda x + B u for piecewise-constant u (Eq. 2 -> Eq. 3)."""
    d = small(P=3, H=2)
    lam, dt, Bc = d["Lambda"].astype(complex), d["Delta"].astype(float), d["Bc"].astype(complex)
    Abar, Bbar = O.zoh_discretize(lam, dt, Bc)
    u0 = np.array([0.7, -1.3])
    x_start = np.array([0.3 - 0.2j, -1.0 + 0.5j, 0.1 + 0.9j])
    for p in range(3):
        sol = solve_ivp(lambda t, x: lam[p] * x + Bc[p] @ u0, (0.0, dt[p]), [x_start[p]],
                        rtol=1e-12, atol=1e-14)
        want = sol.y[0, -1]
        got = Abar[p] * x_start[p] + Bbar[p] @ u0
        assert abs(got - want) < 1e-10


def test_zoh_constant_input_closed_form_and_steady_state():
    d = small(P=5, H=3, T=1)
    lam, dt, Bc = d["Lambda"].astype(complex), d["Delta"].astype(float), d["Bc"].astype(complex)
    Abar, Bbar = O.zoh_discretize(lam, dt, Bc)
    ubar = np.array([0.5, -2.0, 1.25])
    K = 400
    Bu = np.broadcast_to(Bbar @ ubar, (1, K, 5))
    x, _ = O.ssm_scan(Abar, Bu)
    for k in (1, 2, 17, 400):
        want = (np.exp(lam * k * dt) - 1.0) / lam * (Bc @ ubar)
        assert np.allclose(x[0, k - 1], want, rtol=1e-11, atol=1e-13)
        geo = (1 - Abar**k) / (1 - Abar) * (Bbar @ ubar)
        assert np.allclose(x[0, k - 1], geo, rtol=1e-9, atol=1e-12)
    # a strongly damped state has reached -Lambda^{-1} B u
    lam2 = np.array([-40.0 + 3.0j])
    A2, B2 = O.zoh_discretize(lam2, np.array([0.1]), Bc[:1])
    x2, _ = O.ssm_scan(A2, np.broadcast_to(B2 @ ubar, (1, 60, 1)))
    assert np.allclose(x2[0, -1], -(Bc[:1] @ ubar) / lam2, rtol=1e-10)


def test_zoh_small_step_limit_and_no_cancellation():
    lam = np.array([-0.01 + 1e-3j, -1.0 + 3.0j])
    Bc = np.array([[1.0 + 2.0j], [0.5 - 1.0j]])
    for dt in (1e-6, 1e-9):
        Abar, Bbar = O.zoh_discretize(lam, np.full(2, dt), Bc)
        z = lam * dt
        series = dt * (1 + z / 2 + z**2 / 6 + z**3 / 24)      # (e^z - 1)/lam as a power series
        assert np.allclose(Bbar[:, 0], series * Bc[:, 0], rtol=1e-14, atol=0)
        assert np.allclose(Bbar / dt, Bc, rtol=1e-5)


# ---- recurrence / scan ----------------------------------------------------
def test_paper_prefix_identities_and_associativity():
    """Eq. "full_scan": folding the S5 operator gives (Abar^k, x_k) with x_0 = 0."""
    d = small(T=6)
    Abar, Bbar = O.zoh_discretize(d["Lambda"], d["Delta"], d["Bc"])
    Bu = d["u"].astype(float) @ Bbar.T
    x, xT = O.ssm_scan(Abar, Bu)
    rng = random.Random(1)
    for b in range(Bu.shape[0]):
        elems = [(Abar, Bu[b, k]) for k in range(6)]
        acc = elems[0]
        assert np.allclose(acc[1], x[b, 0])
        for k in range(1, 6):
            acc = O.s5_operator(acc, elems[k])
            assert np.allclose(acc[0], Abar ** (k + 1))
            assert np.allclose(acc[1], x[b, k])
        for _ in range(5):
            r = bracket_fold(elems, O.s5_operator, rng)
            assert np.allclose(r[1], xT[b]) and np.allclose(r[0], Abar**6)


def test_bruteforce_unrolled_sum_tiny():
    d = small(T=8, B=1, H=2, P=3)
    Abar, Bbar = O.zoh_discretize(d["Lambda"], d["Delta"], d["Bc"])
    u = d["u"].astype(float)
    y, _, x = O.ssm_layer_fwd(d["Lambda"], d["Delta"], d["Bc"], d["Cc"], d["D"], u)
    Cc, D = d["Cc"].astype(complex), d["D"].astype(float)
    for t in range(1, 9):
        for p in range(3):
            tot = 0j
            for k in range(t):
                a_pow = complex(1.0)
                for _ in range(k):
                    a_pow *= Abar[p]
                for h in range(2):
                    tot += a_pow * Bbar[p, h] * u[0, t - k - 1, h]
            assert abs(tot - x[0, t - 1, p]) < 1e-13
        for h in range(2):
            want = sum((Cc[h, p] * x[0, t - 1, p]).real for p in range(3)) + D[h] * u[0, t - 1, h]
            assert abs(want - y[0, t - 1, h]) < 1e-13


def test_impulse_response():
    d = small(T=9, B=1, H=3, P=4)
    Abar, Bbar = O.zoh_discretize(d["Lambda"], d["Delta"], d["Bc"])
    Cc, D = d["Cc"].astype(complex), d["D"].astype(float)
    for h in range(3):
        u = np.zeros((1, 9, 3))
        u[0, 0, h] = 1.0
        y, _, _ = O.ssm_layer_fwd(d["Lambda"], d["Delta"], d["Bc"], d["Cc"], d["D"], u)
        for t in range(1, 10):
            want = (Cc @ (Abar ** (t - 1) * Bbar[:, h])).real
            if t == 1:
                want = want + D * (np.arange(3) == h)
            assert np.allclose(y[0, t - 1], want, atol=1e-14)


def test_reduces_to_first_order_iir_filter():
    lam, dt = np.array([-0.8 + 0j]), np.array([0.05])
    Bc, Cc, D = np.array([[1.7 + 0j]]), np.array([[1.0 + 0j]]), np.array([0.0])
    u = np.random.default_rng(5).normal(size=(1, 50, 1))
    y, _, _ = O.ssm_layer_fwd(lam, dt, Bc, Cc, D, u)
    a = math.exp(-0.8 * 0.05)
    b = (a - 1.0) / -0.8 * 1.7
    want = lfilter([b], [1.0, -a], u[0, :, 0])
    assert np.allclose(y[0, :, 0], want, rtol=1e-12, atol=1e-14)


def test_structure_linearity_batch_independence_state_permutation():
    d = small(B=3, T=10, H=4, P=6, p_done=0.2, seed=3)
    args = (d["Lambda"], d["Delta"], d["Bc"], d["Cc"], d["D"])
    u = d["u"].astype(float)
    y, _, _ = O.ssm_layer_fwd(*args, u, d["done"])
    u2 = np.random.default_rng(9).normal(size=u.shape)
    y2, _, _ = O.ssm_layer_fwd(*args, u2, d["done"])
    y12, _, _ = O.ssm_layer_fwd(*args, 2.0 * u - 3.0 * u2, d["done"])
    assert np.allclose(y12, 2.0 * y - 3.0 * y2, atol=1e-12)
    yb, _, _ = O.ssm_layer_fwd(*args, u[1:2], d["done"][1:2])
    assert np.allclose(yb[0], y[1], atol=1e-15)
    perm = np.random.default_rng(2).permutation(6)
    yp, _, _ = O.ssm_layer_fwd(d["Lambda"][perm], d["Delta"][perm], d["Bc"][perm],
                               d["Cc"][:, perm], d["D"], u, d["done"])
    assert np.allclose(yp, y, atol=1e-13)


# ---- resets (Sec. IV-A) ----------------------------------------------------
def test_literal_reset_operator_any_bracketing_matches_sequential():
    rng = random.Random(7)
    for seed in range(6):
        d = small(B=2, T=9, p_done=0.35, seed=seed)
        Abar, Bbar = O.zoh_discretize(d["Lambda"], d["Delta"], d["Bc"])
        Bu = d["u"].astype(float) @ Bbar.T
        x, _ = O.ssm_scan(Abar, Bu, d["done"])
        for b in range(2):
            elems = [(Abar, Bu[b, k], int(d["done"][b, k])) for k in range(9)]
            for k in range(9):
                left = elems[0]
                for e in elems[1:k + 1]:
                    left = O.s5_reset_operator(left, e)
                assert np.allclose(left[1], x[b, k])
                r = bracket_fold(elems[:k + 1], O.s5_reset_operator, rng)
                assert np.allclose(r[1], x[b, k])
                assert r[2] == int(d["done"][b, :k + 1].any())   # flag component is the OR


def test_reset_windowed_sum_and_cut_and_concatenate():
    d = small(B=2, T=12, p_done=0.3, seed=11)
    Abar, Bbar = O.zoh_discretize(d["Lambda"], d["Delta"], d["Bc"])
    Bu = d["u"].astype(float) @ Bbar.T
    done = d["done"].copy()
    done[0, 0] = 1            # a flag on the very first step is harmless (x_0 = 0 anyway)
    done[1, 11] = 1
    x, _ = O.ssm_scan(Abar, Bu, done)
    for b in range(2):
        r = None              # steps since the last flagged step (None: none yet)
        start = 0
        for t in range(12):
            if done[b, t]:
                start = t
            want = sum(Abar ** k * Bu[b, t - k] for k in range(t - start + 1))
            assert np.allclose(x[b, t], want)
        # cut at the flags, run the pieces independently from zero, concatenate
        cuts = [0] + [t for t in range(1, 12) if done[b, t]] + [12]
        pieces = [O.ssm_scan(Abar, Bu[b:b + 1, lo:hi])[0] for lo, hi in zip(cuts[:-1], cuts[1:]) if hi > lo]
        assert np.allclose(np.concatenate(pieces, axis=1)[0], x[b])
    xa, _ = O.ssm_scan(Abar, Bu, np.ones((2, 12), np.uint8))
    assert np.allclose(xa, Bu)            # every step flagged: x_t = Bbar u_t


def test_flag_drops_previous_state_but_keeps_current_input():
    """SSM(..., c_{t-1}, x_{t-1}): the flag carried by step t wipes x_{t-1}; u_t still enters."""
    d = small(B=1, T=3, H=2, P=2)
    Abar, Bbar = O.zoh_discretize(d["Lambda"], d["Delta"], d["Bc"])
    Bu = d["u"].astype(float) @ Bbar.T
    done = np.array([[0, 1, 0]], np.uint8)
    x, _ = O.ssm_scan(Abar, Bu, done)
    assert np.allclose(x[0, 1], Bu[0, 1])
    assert np.allclose(x[0, 2], Abar * Bu[0, 1] + Bu[0, 2])
    # non-boolean nonzero values count as set
    x2, _ = O.ssm_scan(Abar, Bu, np.array([[0, 7, 0]], np.uint8))
    assert np.allclose(x2, x)


# ---- initial / final state ---------------------------------------------------
def test_split_invariance_and_x0_response():
    d = small(B=2, T=11, p_done=0.2, seed=4, with_x0=True)
    args = (d["Lambda"], d["Delta"], d["Bc"], d["Cc"], d["D"])
    u = d["u"].astype(float)
    y, xT, x = O.ssm_layer_fwd(*args, u, d["done"], d["x0"])
    for s in (1, 4, 10):
        ya, xs, _ = O.ssm_layer_fwd(*args, u[:, :s], d["done"][:, :s], d["x0"])
        yb, xTb, _ = O.ssm_layer_fwd(*args, u[:, s:], d["done"][:, s:], xs)
        assert np.allclose(np.concatenate([ya, yb], axis=1), y, atol=1e-13)
        assert np.allclose(xTb, xT, atol=1e-13)
        assert np.allclose(xs, x[:, s - 1])
    Abar, _ = O.zoh_discretize(d["Lambda"], d["Delta"], d["Bc"])
    _, _, xz = O.ssm_layer_fwd(*args, np.zeros_like(u), None, d["x0"])
    for t in range(11):
        assert np.allclose(xz[:, t], Abar ** (t + 1) * d["x0"].astype(complex))


def test_flag_on_first_step_beats_x0():
    d = small(B=2, T=4, seed=6, with_x0=True)
    args = (d["Lambda"], d["Delta"], d["Bc"], d["Cc"], d["D"])
    done = np.zeros((2, 4), np.uint8)
    done[0, 0] = 1
    y, _, _ = O.ssm_layer_fwd(*args, d["u"], done, d["x0"])
    y0, _, _ = O.ssm_layer_fwd(*args, d["u"], None, None)
    yx, _, _ = O.ssm_layer_fwd(*args, d["u"], None, d["x0"])
    assert np.allclose(y[0], y0[0]) and np.allclose(y[1], yx[1]) and not np.allclose(y[1], y0[1])


def test_single_step_mode_equals_sequence_mode():
    d = small(B=3, T=6, p_done=0.3, seed=8, with_x0=True)
    args = (d["Lambda"], d["Delta"], d["Bc"], d["Cc"], d["D"])
    y, xT, x = O.ssm_layer_fwd(*args, d["u"], d["done"], d["x0"])
    state = d["x0"]
    for t in range(6):
        state, yt = O.ssm_step(*args, d["u"][:, t], d["done"][:, t], state)
        assert np.allclose(state, x[:, t]) and np.allclose(yt, y[:, t])


# ---- input generator ---------------------------------------------------------
def test_bf16_rounding_helper():
    import torch
    a = np.random.default_rng(0).normal(size=4096).astype(np.float32) * 37.0
    a[:4] = [1.0 + 2**-8, 1.0 + 3 * 2**-8, 0.0, -1e-30]          # two ties: to even
    want = torch.from_numpy(a).to(torch.bfloat16).to(torch.float32).numpy()
    assert np.array_equal(I.round_to_bf16(a), want)


def test_generator_is_seeded_and_shaped():
    d1, d2 = I.draw_layer(I.C1), I.draw_layer(I.C1)
    assert np.array_equal(d1["u"], d2["u"]) and np.array_equal(d1["done"], d2["done"])
    assert d1["u"].shape == (16, 64, 256) and d1["Bc"].shape == (128, 256) and d1["Cc"].shape == (256, 128)
    assert (d1["Lambda"].real <= -0.01 + 1e-7).all() and (d1["Lambda"].real >= -1).all()
    assert (d1["Lambda"].imag >= 0).all() and (d1["Lambda"].imag <= math.pi + 1e-6).all()
    assert (d1["Delta"] >= 1e-3 * (1 - 1e-6)).all() and (d1["Delta"] <= 1e-1 * (1 + 1e-6)).all()
    assert 0 < d1["done"].mean() < 0.05
    assert I.draw_layer(I.C0)["done"] is None
    assert [I.shard_batch(10, r, 4) for r in range(4)] == [(0, 3), (3, 6), (6, 8), (8, 10)]


# ---- conjugate-symmetric parameters ----------------------------------------
def test_conjugate_pairs_fold_into_half_the_states_with_doubled_C():
    """A system whose states come in conjugate pairs (Lambda, B, C and the initial state of state
    p + P/2 are the conjugates of those of state p) has a real output before Re() is taken, and
    Re(C x) over all P states equals Re(2 C x) over the first half: the variant that stores P/2
    states is this layer with C doubled.  Gradients follow by the chain rule (dC_half = 2 x the
    gradient of the doubled C), checked on du and on the first-half parameter gradients."""
    d = small(seed=21, B=2, T=9, H=3, P=4, p_done=0.2, with_x0=True)
    half = {k: d[k] for k in ("Delta", "Lambda", "Bc", "Cc", "x0")}
    Lam = np.concatenate([half["Lambda"], np.conj(half["Lambda"])])
    Dl = np.concatenate([half["Delta"], half["Delta"]])
    Bc = np.concatenate([half["Bc"], np.conj(half["Bc"])], axis=0)
    Cc = np.concatenate([half["Cc"], np.conj(half["Cc"])], axis=1)
    x0 = np.concatenate([half["x0"], np.conj(half["x0"])], axis=1)
    y_full, xT_full, _ = O.ssm_layer_fwd(Lam, Dl, Bc, Cc, d["D"], d["u"], d["done"], x0)
    y_half, xT_half, _ = O.ssm_layer_fwd(half["Lambda"], half["Delta"], half["Bc"], 2.0 * half["Cc"], d["D"], d["u"],
                                         d["done"], half["x0"])
    P = half["Lambda"].shape[0]
    np.testing.assert_allclose(y_full, y_half, rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(xT_full[:, :P], xT_half, rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(xT_full[:, P:], np.conj(xT_half), rtol=1e-12, atol=1e-12)
    g_full = O.ssm_layer_bwd(Lam, Dl, Bc, Cc, d["D"], d["u"], d["done"], x0, d["gy"])
    g_half = O.ssm_layer_bwd(half["Lambda"], half["Delta"], half["Bc"], 2.0 * half["Cc"], d["D"], d["u"], d["done"],
                             half["x0"], d["gy"])
    np.testing.assert_allclose(g_full["du"], g_half["du"], rtol=1e-11, atol=1e-11)
    np.testing.assert_allclose(g_full["dD"], g_half["dD"], rtol=1e-11, atol=1e-11)
    # each parameter of the half system appears twice in the full one (once conjugated): with the
    # convention g = dL/dRe + i dL/dIm the two contributions are g and conj(g) of the pair
    np.testing.assert_allclose(g_full["dB"][:P] + np.conj(g_full["dB"][P:]), g_half["dB"], rtol=1e-10, atol=1e-10)
    np.testing.assert_allclose(g_full["dLambda"][:P] + np.conj(g_full["dLambda"][P:]), g_half["dLambda"], rtol=1e-10,
                               atol=1e-10)
    np.testing.assert_allclose(g_full["dC"][:, :P] + np.conj(g_full["dC"][:, P:]), 2.0 * g_half["dC"], rtol=1e-10,
                               atol=1e-10)
