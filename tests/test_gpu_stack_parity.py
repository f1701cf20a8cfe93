"""Stacked model (SSM -> GELU -> residual -> LayerNorm per layer) on the GPU vs the oracle with
the same storage roundings.

What is compared at the 2e-2 / 1e-4 tolerance is each layer block on the oracle's own inputs
(layer input and incoming gradient taken from the oracle's run), so that only in-layer
arithmetic differs.  End to end, a rounding to the storage type that falls on the other side
of a boundary than in the oracle is amplified by the layers that follow (see
test_oracle_stack_rounding.py).  The end-to-end comparison is therefore only a sanity bound:
n_layers times the tolerance for out and du, twice that for the parameter gradients (sums over
all rows, in which the displaced roundings add up)."""
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
    rnd = I.round_to_bf16 if w.io_dtype == "bf16" else (lambda a: np.asarray(a, np.float32))
    tol = TOL[w.io_dtype]
    out, cache = O.stack_fwd(d["params"], d["ln_weight"], d["ln_bias"], d["u"], d["done"], round_io=rnd)
    du, grads = O.stack_bwd(d["params"], d["ln_weight"], d["ln_bias"], cache, d["done"], d["gy"], round_io=rnd)

    # each block alone, on the oracle's inputs
    g = np.asarray(d["gy"], np.float64)
    for l in range(L - 1, -1, -1):
        sl = slice(l, l + 1)
        o_ref, c_ref = O.stack_fwd(d["params"][sl], d["ln_weight"][sl], d["ln_bias"][sl], cache[l]["u"], d["done"],
                                   round_io=rnd)
        g_ref, gr_ref = O.stack_bwd(d["params"][sl], d["ln_weight"][sl], d["ln_bias"][sl], c_ref, d["done"], g,
                                    round_io=rnd)
        one = {"params": d["params"][sl], "ln_weight": d["ln_weight"][sl], "ln_bias": d["ln_bias"][sl],
               "u": cache[l]["u"].astype(np.float32), "gy": g.astype(np.float32), "done": d["done"]}
        res = harness.run_stack(one, w.io_dtype)
        assert_close(f"layer {l} out", res["out"], o_ref, tol)
        assert_close(f"layer {l} du", res["du"], g_ref, tol)
        for k in GRADS:
            assert_close(f"layer {l} {k}", res["grads"][0][k], gr_ref[0][k], tol)
        g = g_ref

    # the whole stack
    res = harness.run_stack(d, w.io_dtype)
    errs = {"out": assert_close("out", res["out"], out, L * tol), "du": assert_close("du", res["du"], du, L * tol)}
    for l in range(L):
        for k in GRADS:
            errs[f"{k}{l}"] = assert_close(f"stack layer {l} {k}", res["grads"][l][k], grads[l][k], 2 * L * tol)
    print(w.name, {k: f"{v:.1e}" for k, v in errs.items() if v > tol / 10})


def test_c2_stack_of_four_bf16():
    run(I.C2, perturb_ln=False)


def test_c2_stack_of_four_bf16_with_trained_layernorm_affine():
    run(I.C2)


@pytest.mark.parametrize("io", ["f32", "bf16"])
@pytest.mark.parametrize("L,B,T,H,P", [(1, 2, 9, 16, 8), (3, 3, 40, 72, 24), (2, 2, 150, 256, 128)])
def test_small_stacks(io, L, B, T, H, P):
    w = I.Workload("stack", B=B, T=T, H=H, P=P, io_dtype=io, p_done=0.05, n_layers=L, seed=L * 100 + T)
    run(w)
