"""Pins of the oracle's half-GLU gate (Appendix "S5 Sequence Layer"): things the formula and
the mathematics fix, independent of the implementation."""
import math

import numpy as np

from oracle import ssm_oracle as O


def test_zero_weights_halve_the_input():
    # sigmoid(0) = 1/2 whatever GELU gives
    v = np.random.default_rng(0).normal(size=(3, 5, 8))
    out = O.half_glu_fwd(np.zeros((8, 8)), v)
    assert np.allclose(out, 0.5 * v, atol=1e-15)


def test_scalar_case_written_out_by_hand():
    # H = 1: out = v * sigmoid(w * v * Phi(v)), with Phi from math.erf
    for v, w in ((0.7, 1.3), (-1.1, 0.4), (2.5, -0.9)):
        phi = 0.5 * (1.0 + math.erf(v / math.sqrt(2.0)))
        want = v / (1.0 + math.exp(-(w * v * phi)))
        got = O.half_glu_fwd(np.array([[w]]), np.array([[v]]))
        assert abs(got[0, 0] - want) < 1e-15


def test_gate_uses_w_transposed_on_the_gelu_of_the_input():
    # W with a single entry W[i, j]: output feature j is gated by input feature i, the others by 1/2
    rng = np.random.default_rng(1)
    v = rng.normal(size=(4, 6))
    W = np.zeros((6, 6))
    W[2, 5] = 1.7
    out = O.half_glu_fwd(W, v)
    x1 = O.gelu(v)
    want = 0.5 * v
    want[:, 5] = v[:, 5] / (1.0 + np.exp(-1.7 * x1[:, 2]))
    assert np.allclose(out, want, atol=1e-15)


def test_large_positive_and_negative_gates_saturate():
    v = np.array([[3.0, 2.0]])
    W = np.array([[50.0, -50.0], [0.0, 0.0]])      # z = GELU(3) * (50, -50)
    out = O.half_glu_fwd(W, v)
    assert abs(out[0, 0] - 3.0) < 1e-12 and abs(out[0, 1]) < 1e-12


def test_rows_are_independent_and_batch_shape_is_kept():
    rng = np.random.default_rng(2)
    v = rng.normal(size=(2, 3, 5))
    W = rng.normal(size=(5, 5))
    out = O.half_glu_fwd(W, v)
    assert out.shape == v.shape
    assert np.allclose(out[1, 2], O.half_glu_fwd(W, v[1, 2][None])[0], atol=1e-15)


def test_gradients_match_central_differences():
    rng = np.random.default_rng(3)
    v = rng.normal(size=(3, 4, 6))
    W = rng.normal(size=(6, 6)) / np.sqrt(6)
    gout = rng.normal(size=v.shape)
    gv, dW = O.half_glu_bwd(W, v, gout)
    loss = lambda W_, v_: float(np.sum(gout * O.half_glu_fwd(W_, v_)))
    eps = 1e-6
    for idx in [(0, 0, 0), (1, 2, 3), (2, 3, 5)]:
        d = np.zeros_like(v)
        d[idx] = eps
        fd = (loss(W, v + d) - loss(W, v - d)) / (2 * eps)
        assert abs(fd - gv[idx]) < 1e-7 * (1 + abs(fd))
    for idx in [(0, 0), (2, 5), (5, 1)]:
        d = np.zeros_like(W)
        d[idx] = eps
        fd = (loss(W + d, v) - loss(W - d, v)) / (2 * eps)
        assert abs(fd - dW[idx]) < 1e-7 * (1 + abs(fd))


def test_adjoint_identity_in_v():
    # <gout, J dv> = <J^T gout, dv> with J dv from a complex-step-free central difference
    rng = np.random.default_rng(4)
    v = rng.normal(size=(5, 7))
    W = rng.normal(size=(7, 7)) / np.sqrt(7)
    gout = rng.normal(size=v.shape)
    dv = rng.normal(size=v.shape)
    eps = 1e-6
    jv = (O.half_glu_fwd(W, v + eps * dv) - O.half_glu_fwd(W, v - eps * dv)) / (2 * eps)
    gv, _ = O.half_glu_bwd(W, v, gout)
    assert abs(np.sum(gout * jv) - np.sum(gv * dv)) < 1e-7 * (1 + abs(np.sum(gv * dv)))
