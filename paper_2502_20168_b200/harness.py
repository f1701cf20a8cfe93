"""Host-side plumbing around the binding: numpy <-> device buffers, output allocation.

No arithmetic of the method happens here; every step of the layer runs in the
CUDA library.  PyTorch is used only for device memory and streams.
"""
from __future__ import annotations

import numpy as np
import torch

from . import binding as sb

_IO = {"f32": torch.float32, "bf16": torch.bfloat16}


def to_dev(a, dtype=None, device="cuda"):
    if a is None:
        return None
    if isinstance(a, torch.Tensor):      # already a tensor (inputs drawn on the device)
        return (a if dtype is None else a.to(dtype)).to(device).contiguous()
    t = torch.from_numpy(np.ascontiguousarray(a))
    if dtype is not None:
        t = t.to(dtype)
    return t.to(device).contiguous()


def to_np(t):
    if t is None:
        return None
    t = t.detach()
    if t.dtype == torch.bfloat16:
        t = t.float()
    return t.cpu().numpy()


def grad_bucket(P: int, H: int, device="cuda"):
    """One contiguous fp32 buffer holding dLambda[P] c64, dDelta[P], dB[P,H] c64, dC[H,P] c64, dD[H]
    (each segment starts on a 16-byte boundary); returns (bucket, views in that order)."""
    pad = lambda n: (n + 3) // 4 * 4
    sizes = [2 * P, P, 2 * P * H, 2 * H * P, H]          # in floats
    offs = np.concatenate([[0], np.cumsum([pad(n) for n in sizes])])
    bucket = torch.zeros(int(offs[-1]), dtype=torch.float32, device=device)
    seg = [bucket[int(o):int(o) + n] for o, n in zip(offs[:-1], sizes)]
    cplx = lambda t, *shape: torch.view_as_complex(t.view(*shape, 2))
    return bucket, (cplx(seg[0], P), seg[1], cplx(seg[2], P, H), cplx(seg[3], H, P), seg[4])


def allreduce_param_grads(buf, group=None, async_op=False):
    """Sum of the parameter gradients over the ranks of a batch-sharded (data-parallel) run: the one
    exchange such a run has.  Sequences are independent, so every rank's gradients are the sums over
    its own sequences and the full-batch gradients are their sum; y, du and the states stay local.
    One all-reduce over the bucket (NCCL on GPUs; any torch.distributed backend).  With async_op the
    returned handle is waited for before the bucket is read or written again, which lets the exchange
    run under the next step's forward pass."""
    import torch.distributed as dist
    return dist.all_reduce(buf.grad_bucket, op=dist.ReduceOp.SUM, group=group, async_op=async_op)


class GradExchange:
    """Order of the gradient exchange in a batch-sharded training loop.  The layer's backward pass finishes all
    five parameter gradients in its last two kernels (the split-K sums and the adjoint of the discretisation),
    so there is no tail of the backward pass left to hide the exchange under: it is started right after the
    backward call and runs under the next step's forward pass; before the next backward call rewrites the bucket
    the exchange has to be done.  `start()` issues the one all-reduce of the bucket asynchronously; `finish()`
    waits for it (a no-op when none is pending) and must be called before the next backward; a second `start()`
    without `finish()` in between is an error, since the bucket would have been rewritten under the collective."""

    def __init__(self, buf, group=None):
        self.buf, self.group, self.pending = buf, group, None
        self.started = self.finished = 0

    def start(self):
        if self.pending is not None:
            raise RuntimeError("gradient bucket rewritten while its all-reduce was in flight: call finish() first")
        self.pending = allreduce_param_grads(self.buf, group=self.group, async_op=True)
        self.started += 1

    def finish(self):
        if self.pending is not None:
            self.pending.wait()
            self.pending = None
            self.finished += 1


class LayerBuffers:
    """Device copies of one layer's inputs plus preallocated outputs and workspace."""

    def __init__(self, d: dict, io_dtype: str, device="cuda", with_x0=False, with_gxT=False):
        io = _IO[io_dtype]
        B, T, H = d["u"].shape
        P = d["Lambda"].shape[0]
        self.shape = sb.make_shape(B, T, H, P, io_dtype)
        self.io = io
        self.Lambda = to_dev(d["Lambda"].astype(np.complex64), device=device)
        self.Delta = to_dev(d["Delta"].astype(np.float32), device=device)
        self.Bc = to_dev(d["Bc"].astype(np.complex64), device=device)
        self.Cc = to_dev(d["Cc"].astype(np.complex64), device=device)
        self.D = to_dev(d["D"].astype(np.float32), device=device)
        self.u = to_dev(d["u"], io, device)
        self.gy = to_dev(d["gy"], io, device) if d.get("gy") is not None else None
        self.done = to_dev(d.get("done"), torch.uint8, device)
        self.x0 = to_dev(d["x0"].astype(np.complex64), device=device) if with_x0 else None
        self.gxT = to_dev(d["gxT"].astype(np.complex64), device=device) if with_gxT else None
        c64 = dict(dtype=torch.complex64, device=device)
        f32 = dict(dtype=torch.float32, device=device)
        self.y = torch.empty((B, T, H), dtype=io, device=device)
        self.xT = torch.empty((B, P), **c64)
        self.du = torch.empty((B, T, H), dtype=io, device=device)
        # The five parameter gradients are views into one fp32 bucket, so that a data-parallel
        # trainer sums them over the ranks with a single all-reduce and no packing pass.
        self.grad_bucket, (self.dLambda, self.dDelta, self.dB, self.dC, self.dD) = grad_bucket(P, H, device)
        self.dx0 = torch.empty((B, P), **c64)
        self.ws = sb.alloc_workspace(sb.ssm_layer_workspace_bytes(self.shape), device)

    def forward(self, stream=None):
        sb.ssm_layer_fwd(self.shape, self.Lambda, self.Delta, self.Bc, self.Cc, self.D, self.u, self.done,
                         self.x0, self.y, self.xT, self.ws, stream)

    def backward(self, stream=None):
        sb.ssm_layer_bwd(self.shape, self.Lambda, self.Delta, self.Bc, self.Cc, self.D, self.u, self.done,
                         self.x0, self.gy, self.gxT, self.ws, self.du, self.dLambda, self.dDelta, self.dB,
                         self.dC, self.dD, self.dx0, stream)

    def results(self) -> dict:
        return {k: to_np(getattr(self, k)) for k in
                ("y", "xT", "du", "dLambda", "dDelta", "dB", "dC", "dD", "dx0")}


def device_drawn(w, device="cuda") -> dict:
    """A workload's tensors for timing runs: the parameters drawn on the host as always, u, gy and the
    done flags drawn on the device (same distributions; the large tensors never exist on the host).
    Returns a dict that LayerBuffers / StackBuffers accept."""
    from . import inputs as I
    d = I.draw_layer(I.small_variant(w, B=1, T=1))
    g = torch.Generator(device=device)
    g.manual_seed(w.seed)
    io = _IO[w.io_dtype]
    d["u"] = torch.randn((w.B, w.T, w.H), device=device, generator=g).to(io)
    d["gy"] = torch.randn((w.B, w.T, w.H), device=device, generator=g).to(io)
    d["done"] = (torch.rand((w.B, w.T), device=device, generator=g) < w.p_done).to(torch.uint8) if w.p_done > 0 else None
    return d


def run_layer(d: dict, io_dtype: str, with_x0=False, with_gxT=False) -> dict:
    """Forward + backward of one layer on the current CUDA device; returns numpy results."""
    buf = LayerBuffers(d, io_dtype, with_x0=with_x0, with_gxT=with_gxT)
    buf.forward()
    buf.backward()
    sb.ssm_check(buf.ws)
    torch.cuda.synchronize()
    return buf.results()


class StackBuffers:
    """Device copies of a stacked model's inputs plus preallocated outputs and workspace."""

    def __init__(self, d: dict, io_dtype: str, device="cuda"):
        io = _IO[io_dtype]
        B, T, H = d["u"].shape
        P = d["params"][0]["Lambda"].shape[0]
        L = len(d["params"])
        self.shape = sb.make_shape(B, T, H, P, io_dtype)
        self.params, self.grads = [], []
        c64 = dict(dtype=torch.complex64, device=device)
        f32 = dict(dtype=torch.float32, device=device)
        for l in range(L):
            q = d["params"][l]
            self.params.append({
                "Lambda": to_dev(q["Lambda"].astype(np.complex64), device=device),
                "Delta": to_dev(q["Delta"].astype(np.float32), device=device),
                "Bc": to_dev(q["Bc"].astype(np.complex64), device=device),
                "Cc": to_dev(q["Cc"].astype(np.complex64), device=device),
                "D": to_dev(q["D"].astype(np.float32), device=device),
                "ln_weight": to_dev(np.asarray(d["ln_weight"][l], np.float32), device=device),
                "ln_bias": to_dev(np.asarray(d["ln_bias"][l], np.float32), device=device)})
            self.grads.append({
                "dLambda": torch.empty(P, **c64), "dDelta": torch.empty(P, **f32),
                "dB": torch.empty((P, H), **c64), "dC": torch.empty((H, P), **c64), "dD": torch.empty(H, **f32),
                "dln_weight": torch.empty(H, **f32), "dln_bias": torch.empty(H, **f32)})
        self.u = to_dev(d["u"], io, device)
        self.gout = to_dev(d["gy"], io, device)
        self.done = to_dev(d.get("done"), torch.uint8, device)
        self.out = torch.empty((B, T, H), dtype=io, device=device)
        self.du = torch.empty((B, T, H), dtype=io, device=device)
        self.ws = sb.alloc_workspace(sb.ssm_stack_workspace_bytes(self.shape, L), device)

    def forward(self, stream=None):
        sb.ssm_stack_fwd(self.shape, self.params, self.u, self.done, self.out, self.ws, stream)

    def backward(self, stream=None):
        sb.ssm_stack_bwd(self.shape, self.params, self.u, self.done, self.gout, self.ws, self.du, self.grads, stream)

    def results(self) -> dict:
        return {"out": to_np(self.out), "du": to_np(self.du),
                "grads": [{k: to_np(v) for k, v in g.items()} for g in self.grads]}


def run_stack(d: dict, io_dtype: str) -> dict:
    buf = StackBuffers(d, io_dtype)
    buf.forward()
    buf.backward()
    sb.ssm_check(buf.ws)
    torch.cuda.synchronize()
    return buf.results()
