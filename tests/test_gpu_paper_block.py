"""The paper's sequence block (Appendix "S5 Sequence Layer": SSM layer, then the half-GLU gate on its
output) at the sizes of the paper's vision task (two blocks, deterministic state 1024, SSM state 512,
batches of 32 x 128 steps; hyper-parameter tables of the appendix), bf16 I/O, against the oracle's
composition of ssm_layer_* and half_glu_*.

What is compared, and how:
 * every block alone on the oracle's own block inputs (block input and incoming gradient taken from
   the oracle's run, which rounds to bf16 exactly the tensors that the CUDA path stores as bf16: the
   layer output, the block output and their gradients): the block's output and its input gradient
   elementwise at the bf16 tolerance;
 * the parameter gradients of a block (sums over all 4096 rows) against the tolerance times the
   scale of the gradient, max |err| <= tol (1 + max |ref|): the layer output that the gate reads is
   a bf16 tensor, the CUDA path's copy of it differs from the oracle's by one bf16 unit wherever the
   two evaluations fall on different sides of a rounding boundary, and those units add up in the
   sums like any other noise of relative size 2^-9, which elements far below the gradient's scale
   cannot absorb.  (The layer and the gate are each held to the elementwise tolerance on identical
   inputs by their own tests, the gate at this size below.)  The elementwise figures are printed;
 * the two blocks end to end: printed, and asserted at the same bounds."""
import numpy as np
import pytest

from oracle import ssm_oracle as O
from paper_2502_20168_b200 import inputs as I
from tests.util import TOL, assert_close, worst

pytestmark = pytest.mark.gpu
PARAMS = ("Lambda", "Delta", "Bc", "Cc", "D")
GRADS = ("dLambda", "dDelta", "dB", "dC", "dD")
rnd = I.round_to_bf16


def _r(a):
    return rnd(a).astype(np.float64)


def oracle_blocks(params, Ws, u, done, gout):
    """Forward and backward of the chain of blocks in float64 with bf16 roundings at the tensors the
    CUDA path stores as bf16.  Returns per block: input, output, incoming gradient, du, gradients."""
    n = len(params)
    ins, vs, outs = [], [], []
    x = np.asarray(u, np.float64)
    for p, W in zip(params, Ws):
        y, _, _ = O.ssm_layer_fwd(*(p[k] for k in PARAMS), x, done, None)
        v = _r(y)
        o = _r(O.half_glu_fwd(W, v))
        ins.append(x), vs.append(v), outs.append(o)
        x = o
    g = np.asarray(gout, np.float64)
    gins, dus, grads = [None] * n, [None] * n, [None] * n
    for l in range(n - 1, -1, -1):
        gins[l] = g
        gv, dW = O.half_glu_bwd(Ws[l], vs[l], g)
        r = O.ssm_layer_bwd(*(params[l][k] for k in PARAMS), ins[l], done, None, _r(gv))
        grads[l] = {k: r[k] for k in GRADS}
        grads[l]["dW"] = dW
        dus[l] = _r(r["du"])
        g = dus[l]
    return ins, outs, gins, dus, grads


class GpuBlocks:
    """The chain of blocks on the GPU through the C ABI: per block one layer workspace and one gate workspace."""

    def __init__(self, w, params, Ws, done):
        import torch
        from paper_2502_20168_b200 import binding as sb, harness
        self.sb, self.torch = sb, torch
        self.shape = sb.make_shape(w.B, w.T, w.H, w.P, "bf16")
        zero = np.zeros((w.B, w.T, w.H), np.float32)
        self.layers = [harness.LayerBuffers(dict(p, u=zero, gy=zero, done=done), "bf16") for p in params]
        self.Ws = [harness.to_dev(W) for W in Ws]
        self.dWs = [torch.empty_like(W) for W in self.Ws]
        self.gws = [sb.alloc_workspace(sb.ssm_glu_workspace_bytes(self.shape)) for _ in Ws]
        self.outs = [torch.empty_like(self.layers[0].y) for _ in Ws]

    def forward(self, first, last, u):
        sb = self.sb
        x = u
        for l in range(first, last + 1):
            L = self.layers[l]
            L.u = x
            L.forward()
            sb.ssm_glu_fwd(self.shape, self.Ws[l], L.y, self.outs[l], self.gws[l])
            x = self.outs[l]
        return x

    def backward(self, first, last, gout):
        sb = self.sb
        g = gout
        for l in range(last, first - 1, -1):
            L = self.layers[l]
            L.gy = self.torch.empty_like(L.y)
            sb.ssm_glu_bwd(self.shape, self.Ws[l], L.y, g, self.gws[l], L.gy, self.dWs[l])
            L.backward()
            g = L.du
        for l in range(first, last + 1):
            sb.ssm_check(self.layers[l].ws)
            sb.ssm_check(self.gws[l])
        return g

    def grads(self, l):
        from paper_2502_20168_b200 import harness
        r = self.layers[l].results()
        out = {k: r[k] for k in GRADS}
        out["dW"] = harness.to_np(self.dWs[l])
        return out


def scale_err(got, ref):
    return float(np.max(np.abs(got - ref)) / (1.0 + np.max(np.abs(ref))))


def test_two_blocks_at_the_vision_sizes_bf16():
    from paper_2502_20168_b200 import harness
    import torch
    w = I.small_variant(I.PAPER_VISION, n_layers=2)
    d = I.draw_layer(w)
    params = d["params"]
    Ws = [I.draw_glu(I.small_variant(w, seed=w.seed + 10 * l))["W"] for l in range(2)]
    tol = TOL["bf16"]
    ins, outs, gins, dus, grads = oracle_blocks(params, Ws, d["u"], d["done"], d["gy"])
    gpu = GpuBlocks(w, params, Ws, d["done"])
    dev = lambda a: harness.to_dev(np.asarray(a, np.float32), torch.bfloat16)

    report = {}
    for l in (1, 0):      # each block alone on the oracle's inputs
        out = gpu.forward(l, l, dev(ins[l]))
        du = gpu.backward(l, l, dev(gins[l]))
        report[f"block{l} out"] = assert_close(f"block {l} out", harness.to_np(out), outs[l], tol)
        report[f"block{l} du"] = assert_close(f"block {l} du", harness.to_np(du), dus[l], tol)
        for k, got in gpu.grads(l).items():
            s = scale_err(got, grads[l][k])
            assert s <= tol, f"block {l} {k}: max |err| / (1 + max |ref|) = {s:.3e}"
            report[f"block{l} {k}"] = f"{s:.1e} of scale, {worst(got, grads[l][k]):.1e} elementwise"
    # both blocks end to end
    out = gpu.forward(0, 1, dev(d["u"]))
    du = gpu.backward(0, 1, dev(d["gy"]))
    report["e2e out"] = assert_close("end to end out", harness.to_np(out), outs[1], tol)
    report["e2e du"] = assert_close("end to end du", harness.to_np(du), dus[0], tol)
    for l in (0, 1):
        for k, got in gpu.grads(l).items():
            s = scale_err(got, grads[l][k])
            assert s <= tol, f"end to end, block {l} {k}: {s:.3e}"
            report[f"e2e block{l} {k}"] = f"{s:.1e} of scale, {worst(got, grads[l][k]):.1e} elementwise"
    print("paper block, vision sizes:", report)


def test_gate_at_the_vision_sizes_bf16():
    """The gate alone at H = 1024 on 32 x 128 rows, identical inputs: elementwise at the bf16 tolerance."""
    from tests.test_gpu_half_glu import _run
    _run(I.Workload("glu_vision", B=32, T=128, H=1024, P=8, io_dtype="bf16", seed=6))
