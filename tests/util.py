"""Helpers shared by the GPU parity tests: run the oracle on a drawn workload, compare."""
import numpy as np

from oracle import ssm_oracle as O

TOL = {"f32": 1e-4, "bf16": 2e-2}     # max |err| <= tol * (1 + |ref|), elementwise


def oracle_layer(d, with_x0=False, with_gxT=False):
    x0 = d["x0"] if with_x0 else None
    gxT = d["gxT"] if with_gxT else None
    y, xT, x = O.ssm_layer_fwd(d["Lambda"], d["Delta"], d["Bc"], d["Cc"], d["D"], d["u"], d["done"], x0)
    g = O.ssm_layer_bwd(d["Lambda"], d["Delta"], d["Bc"], d["Cc"], d["D"], d["u"], d["done"], x0, d["gy"], gxT)
    g.update(y=y, xT=xT, x=x)
    return g


def worst(got, ref):
    """max over elements of |got - ref| / (1 + |ref|)."""
    got = np.asarray(got)
    ref = np.asarray(ref)
    assert got.shape == ref.shape, (got.shape, ref.shape)
    assert np.isfinite(got).all()
    return float(np.max(np.abs(got.astype(ref.dtype) - ref) / (1.0 + np.abs(ref)))) if ref.size else 0.0


def assert_close(name, got, ref, tol):
    w = worst(got, ref)
    assert w <= tol, f"{name}: max |err|/(1+|ref|) = {w:.3e} > {tol:g}"
    return w


def compare_layer(res, ref, io_dtype, keys=("y", "xT", "du", "dLambda", "dDelta", "dB", "dC", "dD")):
    tol = TOL[io_dtype]
    return {k: assert_close(k, res[k], ref[k], tol) for k in keys}
