"""Stacked model (SSM -> GELU -> residual -> LayerNorm per layer) on the GPU against the float64
oracle, end to end: the stack's output, the input gradient and every layer's parameter gradients
at the tolerance of the I/O type, elementwise.  The oracle runs in float64 throughout (no storage
rounding anywhere); the CUDA path keeps what passes between the layers in fp32 and rounds only the
stack's own output and input gradient to the I/O type."""
import numpy as np
import pytest

from oracle import ssm_oracle as O
from paper_2502_20168_b200 import inputs as I
from tests.util import TOL, assert_close

pytestmark = pytest.mark.gpu
GRADS = ("dLambda", "dDelta", "dB", "dC", "dD", "dln_weight", "dln_bias")


def draw(w, perturb_ln):
    d = I.draw_layer(w)
    if w.n_layers == 1:
        d["params"] = [{k: d[k] for k in ("Lambda", "Delta", "Bc", "Cc", "D")}]
        d["ln_weight"] = [np.ones(w.H, np.float32)]
        d["ln_bias"] = [np.zeros(w.H, np.float32)]
    if perturb_ln:      # LayerNorm affine away from its (1, 0) initial values
        rng = np.random.default_rng(w.seed + 50)
        d["ln_weight"] = [(1.0 + 0.1 * rng.normal(size=w.H)).astype(np.float32) for _ in range(w.n_layers)]
        d["ln_bias"] = [(0.1 * rng.normal(size=w.H)).astype(np.float32) for _ in range(w.n_layers)]
    return d


def run(w, perturb_ln=True):
    from paper_2502_20168_b200 import harness
    d = draw(w, perturb_ln)
    L = w.n_layers
    tol = TOL[w.io_dtype]
    out, cache = O.stack_fwd(d["params"], d["ln_weight"], d["ln_bias"], d["u"], d["done"])
    du, grads = O.stack_bwd(d["params"], d["ln_weight"], d["ln_bias"], cache, d["done"], d["gy"])
    res = harness.run_stack(d, w.io_dtype)
    errs = {"out": assert_close("out", res["out"], out, tol), "du": assert_close("du", res["du"], du, tol)}
    for l in range(L):
        for k in GRADS:
            errs[f"{k}[{l}]"] = assert_close(f"layer {l} {k}", res["grads"][l][k], grads[l][k], tol)
    print(w.name, {k: f"{v:.1e}" for k, v in errs.items()})
    return errs


def test_c2_stack_of_four_bf16():
    run(I.C2, perturb_ln=False)


def test_c2_stack_of_four_bf16_with_trained_layernorm_affine():
    run(I.C2)


@pytest.mark.parametrize("io", ["f32", "bf16"])
@pytest.mark.parametrize("L,B,T,H,P", [(1, 2, 9, 16, 8), (3, 3, 40, 72, 24), (2, 2, 150, 256, 128)])
def test_small_stacks(io, L, B, T, H, P):
    w = I.Workload("stack", B=B, T=T, H=H, P=P, io_dtype=io, p_done=0.05, n_layers=L, seed=L * 100 + T)
    run(w)
