"""Float64 CPU oracle for the S5 state-space layer of the paper's world model.

TEST INFRASTRUCTURE ONLY.  This file is the slow, plain statement of what the
layer computes; it exists so that the CUDA library can be checked against it.
Only the test-suite, the smoke check and the benchmark's CPU-baseline leg may
import it.  It shares no code with the CUDA path and never falls back to it.

What it follows (all in float64 / complex128, one time step after the other):

* Sec. III-B, Eq. 2-3: the linear system dx/dt = A x + B u, y = C x + D u with a
  diagonal complex A = diag(Lambda), sampled with a fixed step Delta:
      x_t = Abar x_{t-1} + Bbar u_t,     y_t = Re(C x_t) + D * u_t.
  The paper says only that (Abar, Bbar) are functions of the continuous
  matrices; the zero-order hold is used here:
      Abar = exp(Lambda Delta),  Bbar = Lambda^{-1} (Abar - 1) B,  C and D unchanged.
* Sec. III-B, Eq. "scan"/"associative"/"sequence_scan"/"full_scan": the parallel
  scan reaches exactly the sequential recurrence with x_0 = 0, so the recurrence
  IS the definition; `s5_operator` is kept only to test that claim.
* Sec. IV-A, Eq. "sequence_scan_reset"/"associative_reset": an element whose
  done flag (1 - c_k) is set discards everything before it, i.e. the state is
  zeroed before that step's update and the step's own input still enters.
* Sec. IV-A Eq. "wm" and Sec. IV-B Eq. "imaginationproc": the sequence model is
  also called one step at a time with an explicit previous state, hence the
  optional initial state x0 and the returned final state xT.

Gradient convention for complex quantities under a real loss L:
    g_z := dL/dRe(z) + i dL/dIm(z).

Pins: every function here is pinned by tests that run without a GPU (closed
forms, brute-force unrolling, the paper's prefix identities, the literal
operators under random bracketings, a textbook IIR filter, finite differences,
the adjoint identity and an independent autograd derivation).
"""
from __future__ import annotations

import numpy as np
from scipy.special import erf as _erf

C128 = np.complex128
F64 = np.float64


# --------------------------------------------------------------------------
# Discretisation (Sec. III-B, Eq. 3; zero-order hold)
# --------------------------------------------------------------------------
def _expm1_complex(z: np.ndarray) -> np.ndarray:
    """exp(z) - 1 without cancellation for small |z|."""
    a, b = z.real, z.imag
    # e^a cos b - 1 = expm1(a) cos b + (cos b - 1),  cos b - 1 = -2 sin^2(b/2)
    re = np.expm1(a) * np.cos(b) - 2.0 * np.sin(0.5 * b) ** 2
    im = np.exp(a) * np.sin(b)
    return re + 1j * im


def zoh_discretize(Lambda, Delta, Bc):
    """Abar[P] = exp(Lambda Delta);  Bbar[P,H] = ((Abar - 1) / Lambda) * B   (row-wise)."""
    Lambda = np.asarray(Lambda, C128)
    Delta = np.asarray(Delta, F64)
    Bc = np.asarray(Bc, C128)
    z = Lambda * Delta
    Abar = np.exp(z)
    gamma = _expm1_complex(z) / Lambda
    return Abar, gamma[:, None] * Bc


def zoh_discretize_bwd(Lambda, Delta, Bc, gAbar, gBbar):
    """Adjoint of `zoh_discretize`: returns (dLambda[P], dDelta[P], dB[P,H]).

    With z = Lambda Delta, gamma = (e^z - 1)/Lambda:
      dAbar/dLambda = Delta Abar,  dAbar/dDelta = Lambda Abar,
      dgamma/dLambda = (Delta Abar Lambda - (Abar - 1)) / Lambda^2,  dgamma/dDelta = Abar.
    All maps are holomorphic in Lambda, so g_Lambda = conj(d./dLambda) g_. ; Delta is
    real, so g_Delta = Re(conj(d./dDelta) g_.).
    """
    Lambda = np.asarray(Lambda, C128)
    Delta = np.asarray(Delta, F64)
    Bc = np.asarray(Bc, C128)
    gAbar = np.asarray(gAbar, C128)
    gBbar = np.asarray(gBbar, C128)
    z = Lambda * Delta
    Abar = np.exp(z)
    em1 = _expm1_complex(z)
    gamma = em1 / Lambda
    dB = np.conj(gamma)[:, None] * gBbar
    ggamma = np.sum(np.conj(Bc) * gBbar, axis=1)
    dgamma_dL = (Delta * Abar * Lambda - em1) / Lambda**2
    dLambda = np.conj(Delta * Abar) * gAbar + np.conj(dgamma_dL) * ggamma
    dDelta = (np.conj(Lambda * Abar) * gAbar).real + (np.conj(Abar) * ggamma).real
    return dLambda, dDelta, dB


# --------------------------------------------------------------------------
# The recurrence (Sec. III-B Eq. 3 / "full_scan"; resets: Sec. IV-A)
# --------------------------------------------------------------------------
def ssm_scan(Abar, Bu, done=None, x0=None):
    """x_t = (done_t ? 0 : Abar * x_{t-1}) + Bu_t for t = 1..T, per sequence and state.

    Abar[P], Bu[B,T,P] complex, done[B,T] (nonzero = the episode ended before step t,
    so the carried state is dropped), x0[B,P] or None (= 0).  Returns (x[B,T,P], xT[B,P]).
    """
    Abar = np.asarray(Abar, C128)
    Bu = np.asarray(Bu, C128)
    Bsz, T, P = Bu.shape
    x = np.empty((Bsz, T, P), C128)
    state = np.zeros((Bsz, P), C128) if x0 is None else np.array(x0, C128)
    for t in range(T):
        if done is not None:
            state = np.where(np.asarray(done)[:, t, None] != 0, 0.0, state)
        state = Abar[None, :] * state + Bu[:, t, :]
        x[:, t, :] = state
    return x, state.copy()


def ssm_scan_bwd(Abar, x, done, x0, gx, gxT=None):
    """Adjoint of `ssm_scan` w.r.t. (Bu, Abar, x0), given g_x[B,T,P] and optional g_xT[B,P].

    s_t = g_x,t + (1 - done_{t+1}) conj(Abar) s_{t+1}   (s_{T+1} := g_xT or 0);
    gBu_t = s_t;  gAbar = sum_{b,t} (1 - done_t) s_t conj(x_{t-1});
    gx0 = (1 - done_1) conj(Abar) s_1.
    """
    Abar = np.asarray(Abar, C128)
    x = np.asarray(x, C128)
    gx = np.asarray(gx, C128)
    Bsz, T, P = gx.shape
    s_all = np.empty((Bsz, T, P), C128)
    gAbar = np.zeros(P, C128)
    carry = np.zeros((Bsz, P), C128) if gxT is None else np.array(gxT, C128)
    x_init = np.zeros((Bsz, P), C128) if x0 is None else np.asarray(x0, C128)
    for t in range(T - 1, -1, -1):
        s = gx[:, t, :] + carry
        s_all[:, t, :] = s
        keep = 1.0 if done is None else (np.asarray(done)[:, t, None] == 0).astype(F64)
        x_prev = x[:, t - 1, :] if t > 0 else x_init
        gAbar += np.sum(keep * s * np.conj(x_prev), axis=0)
        carry = keep * np.conj(Abar)[None, :] * s
    return s_all, gAbar, carry


def ssm_layer_fwd(Lambda, Delta, Bc, Cc, D, u, done=None, x0=None):
    """y[B,T,H], xT[B,P], x[B,T,P] of the discretised diagonal SSM (Eq. 3 with resets)."""
    u = np.asarray(u, F64)
    Cc = np.asarray(Cc, C128)
    D = np.asarray(D, F64)
    Abar, Bbar = zoh_discretize(Lambda, Delta, Bc)
    Bu = u @ Bbar.T                      # Bu[b,t,p] = sum_h Bbar[p,h] u[b,t,h]
    x, xT = ssm_scan(Abar, Bu, done, x0)
    y = (x @ Cc.T).real + D * u          # y[b,t,h] = Re sum_p C[h,p] x[b,t,p] + D_h u[b,t,h]
    return y, xT, x


def ssm_layer_bwd(Lambda, Delta, Bc, Cc, D, u, done, x0, gy, gxT=None):
    """Gradients of L = sum(gy * y) + Re sum(conj(gxT) xT) w.r.t. every input.

    Returns dict(du, dLambda, dDelta, dB, dC, dD, dx0).
    """
    u = np.asarray(u, F64)
    gy = np.asarray(gy, F64)
    Cc = np.asarray(Cc, C128)
    D = np.asarray(D, F64)
    Bsz, T, H = u.shape
    Abar, Bbar = zoh_discretize(Lambda, Delta, Bc)
    x, _ = ssm_scan(Abar, u @ Bbar.T, done, x0)
    # y = Re(C x) + D u
    gx = gy @ np.conj(Cc)                                # [B,T,P]
    P = x.shape[-1]
    dC = gy.reshape(-1, H).T @ np.conj(x).reshape(-1, P)      # dC[h,p] = sum_{b,t} gy[b,t,h] conj(x[b,t,p])
    dD = np.sum(gy * u, axis=(0, 1))
    # x = scan(Abar, Bu)
    s, gAbar, gx0 = ssm_scan_bwd(Abar, x, done, x0, gx, gxT)
    # Bu = Bbar u  (u real)
    du = D * gy + (s @ np.conj(Bbar)).real
    gBbar = s.reshape(-1, P).T @ u.reshape(-1, H)             # gBbar[p,h] = sum_{b,t} s[b,t,p] u[b,t,h]
    dLambda, dDelta, dB = zoh_discretize_bwd(Lambda, Delta, Bc, gAbar, gBbar)
    return {"du": du, "dLambda": dLambda, "dDelta": dDelta, "dB": dB, "dC": dC,
            "dD": dD, "dx0": gx0}


def ssm_step(Lambda, Delta, Bc, Cc, D, u_t, done_t, x_prev):
    """One call of the sequence model, x_t, y_t = SSM(u_t, done_t, x_{t-1}) (Eq. "wm")."""
    Abar, Bbar = zoh_discretize(Lambda, Delta, Bc)
    x_prev = np.asarray(x_prev, C128)
    if done_t is not None:
        x_prev = np.where(np.asarray(done_t)[:, None] != 0, 0.0, x_prev)
    u_t = np.asarray(u_t, F64)
    x_t = Abar[None, :] * x_prev + u_t @ Bbar.T
    y_t = (x_t @ np.asarray(Cc, C128).T).real + np.asarray(D, F64) * u_t
    return x_t, y_t


# --------------------------------------------------------------------------
# The paper's scan operators, literally (used only to test the claims above)
# --------------------------------------------------------------------------
def s5_operator(ai, aj):
    """Eq. "associative": (a_i . a_j) = (a_j,a * a_i,a,  a_j,a * a_i,b + a_j,b), diagonal a."""
    return (aj[0] * ai[0], aj[0] * ai[1] + aj[1])


def s5_reset_operator(ai, aj):
    """Eq. "associative_reset": the third component is the done flag 1 - c."""
    if aj[2] == 0:
        return (aj[0] * ai[0], aj[0] * ai[1] + aj[1], ai[2])
    return (aj[0], aj[1], aj[2])


# --------------------------------------------------------------------------
# Stacked sequence model: out = LayerNorm(u + GELU(SSM(u))) per layer
# --------------------------------------------------------------------------
LN_EPS = 1e-5


def gelu(v):
    """Exact GELU, v * Phi(v) (the appendix calls it the standard GELU)."""
    return 0.5 * v * (1.0 + _erf(v / np.sqrt(2.0)))


def gelu_grad(v):
    return 0.5 * (1.0 + _erf(v / np.sqrt(2.0))) + v * np.exp(-0.5 * v * v) / np.sqrt(2.0 * np.pi)


# --------------------------------------------------------------------------
# Half-GLU gate of the S5 sequence layer (Appendix "S5 Sequence Layer")
# --------------------------------------------------------------------------
def half_glu_fwd(W, v):
    """x1 = GELU(v);  out = v * sigmoid(W^T x1), row by row (v: [..., H], W: [H, H]).

    Appendix "S5 Sequence Layer": the gate's argument is the linear layer W applied to the
    GELU of the gate's input, (W^T x1)_j = sum_i W[i, j] x1_i; the input itself is what gets
    gated.  No bias (the appendix names only the weights W)."""
    v = np.asarray(v, F64)
    W = np.asarray(W, F64)
    z = gelu(v) @ W
    return v / (1.0 + np.exp(-z))


def half_glu_bwd(W, v, gout):
    """Gradients of L = sum(gout * out) for out = half_glu_fwd(W, v): (gv, dW)."""
    v = np.asarray(v, F64)
    W = np.asarray(W, F64)
    gout = np.asarray(gout, F64)
    x1 = gelu(v)
    s = 1.0 / (1.0 + np.exp(-(x1 @ W)))
    gz = gout * v * s * (1.0 - s)
    gv = gout * s + (gz @ W.T) * gelu_grad(v)
    H = v.shape[-1]
    dW = x1.reshape(-1, H).T @ gz.reshape(-1, H)
    return gv, dW


def layernorm_fwd(z, weight, bias):
    mu = z.mean(axis=-1, keepdims=True)
    var = ((z - mu) ** 2).mean(axis=-1, keepdims=True)
    rstd = 1.0 / np.sqrt(var + LN_EPS)
    zhat = (z - mu) * rstd
    return zhat * weight + bias, zhat, rstd


def layernorm_bwd(gout, zhat, rstd, weight):
    gw = np.sum(gout * zhat, axis=tuple(range(gout.ndim - 1)))
    gb = np.sum(gout, axis=tuple(range(gout.ndim - 1)))
    gzhat = gout * weight
    gz = rstd * (gzhat - gzhat.mean(axis=-1, keepdims=True)
                 - zhat * (gzhat * zhat).mean(axis=-1, keepdims=True))
    return gz, gw, gb


def _identity(a):
    return a


def stack_fwd(params, ln_weight, ln_bias, u, done=None, round_io=_identity):
    """n layers of  v = SSM(u);  out = LayerNorm(u + GELU(v)) * w + b.

    `round_io` (identity by default = all float64) models a storage precision for the
    tensors that are a layer's inputs and outputs: the SSM output v and the block output.
    It exists to study what such roundings do to the gradients; the CUDA path keeps these
    tensors in fp32 and is compared with the default.  Returns (out, cache).
    """
    cache = []
    act = np.asarray(u, F64)
    for p, w, b in zip(params, ln_weight, ln_bias):
        y, _, _ = ssm_layer_fwd(p["Lambda"], p["Delta"], p["Bc"], p["Cc"], p["D"], act, done, None)
        v = round_io(y).astype(F64)
        z = act + gelu(v)
        out, zhat, rstd = layernorm_fwd(z, np.asarray(w, F64), np.asarray(b, F64))
        cache.append({"u": act, "v": v, "zhat": zhat, "rstd": rstd})
        act = round_io(out).astype(F64)
    return act, cache


def stack_bwd(params, ln_weight, ln_bias, cache, done, gout, round_io=_identity):
    """Backward of `stack_fwd` (rounding treated as identity in the derivative).

    Per layer, top down:  gz = LN'(gout);  gv = round(gz * GELU'(v)) is the SSM layer's
    incoming gradient;  the gradient handed to the layer below is round(gz + du_ssm): only what
    enters or leaves a layer is rounded, nothing inside it.
    Returns (du, [per-layer dict(dLambda, dDelta, dB, dC, dD, dln_weight, dln_bias)]).
    """
    g = np.asarray(gout, F64)
    grads = [None] * len(params)
    for l in range(len(params) - 1, -1, -1):
        p, c = params[l], cache[l]
        gz, gw, gb = layernorm_bwd(g, c["zhat"], c["rstd"], np.asarray(ln_weight[l], F64))
        gv = round_io(gz * gelu_grad(c["v"])).astype(F64)
        r = ssm_layer_bwd(p["Lambda"], p["Delta"], p["Bc"], p["Cc"], p["D"], c["u"], done, None, gv)
        g = round_io(gz + r["du"]).astype(F64)
        grads[l] = {k: r[k] for k in ("dLambda", "dDelta", "dB", "dC", "dD")}
        grads[l]["dln_weight"] = gw
        grads[l]["dln_bias"] = gb
    return g, grads
