#!/usr/bin/env python
"""Benchmark of the SSM layer forward + backward (timesteps per second) on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl reference]

One step is one forward + backward pass of the layer over one synthetic batch.  With N > 1
(launched by torch.distributed.run) every rank runs the same workload on its own seeded
batch: sequences are independent, so the path shards over the batch with no collective on
the data path; the reported value is the sum over ranks divided by the slowest rank's time.
Prints one JSON line on rank 0.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

from paper_2502_20168_b200 import inputs as I  # noqa: E402

METRIC = "ssm_layer_fwd_bwd_timesteps_per_sec"
UNIT = "timesteps/s"
DEFAULT_WORKLOAD = "c4_sweep_T1024_bf16"
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}

# Algorithmic work of each internal stage per timestep (one (b,t) row; s = bytes of an I/O element):
# (flops, bytes).  A projection is a real GEMM with K*N = 2*H*P per row; a scan moves 16 or 24 bytes
# per state and step.  A stage that is both (projection and scan in one kernel) names its flops and the
# bytes it has to move (operand in, state planes in / out); the roofline that bounds it is the one whose
# floor (work / measured peak) is the longer time.
STAGE_MODEL = {
    "gemm_Bu_scan_fwd": (lambda H, P, s: 4.0 * H * P, lambda H, P, s: H * s + 8.0 * P),      # u in, x planes out
    "gemm_gx_scan_bwd": (lambda H, P, s: 4.0 * H * P, lambda H, P, s: H * s + 16.0 * P),     # gy, x planes in, s planes out
    "gemm_Bu": (lambda H, P, s: 4.0 * H * P, None),
    "scan_fwd": (None, lambda H, P, s: 16.0 * P),
    "gemm_y": (lambda H, P, s: 4.0 * H * P, None),
    "gemm_gx": (lambda H, P, s: 4.0 * H * P, None),
    "scan_bwd": (None, lambda H, P, s: 24.0 * P),
    "gemm_du": (lambda H, P, s: 4.0 * H * P, None),
    "gemm_gBbar": (lambda H, P, s: 4.0 * H * P, None),
    "gemm_gC": (lambda H, P, s: 4.0 * H * P, None),
}


# DRAM bytes per timestep seen by ncu (dram__bytes_read.sum + dram__bytes_write.sum, or dram__bytes.sum.per_second x
# duration; summaries under profiles/), captured on c4_sweep_T1024_bf16 cut down to B = 128 (131072 rows) and divided
# by those rows: every kernel's traffic is proportional to the rows it processes, so a launch of the full workload
# moves this figure times its timesteps.  They hold for H = 512, P = 256, bf16 I/O, T = 1024; an entry is None where
# no capture of the kernel as it stands exists.
NCU_TRAFFIC_PER_TIMESTEP = {
    "gemm_Bu_scan_fwd": 349.9e6 / 131072,
    "gemm_gx_scan_bwd": 644.7e6 / 131072,
    "gemm_y": 379.7e6 / 131072,
    "gemm_du": 546.9e6 / 131072,
    "gemm_gBbar": 406.5e6 / 131072,
    "gemm_gC": 406.6e6 / 131072,
    "scan_fwd": None,
    "scan_bwd": None,
    "gemm_Bu": None,
    "gemm_gx": None,
}


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return p, "measured"
    return dict(FALLBACK_PEAKS), "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons through NVML (read-only queries) from a thread
    while the timed region runs; falls back to one nvidia-smi query loop if NVML is missing."""

    REASONS = (("hw_slowdown", 0x8), ("sw_thermal_slowdown", 0x20), ("hw_thermal_slowdown", 0x40),
               ("sw_power_cap", 0x4), ("applications_clocks_setting", 0x2), ("sync_boost", 0x10),
               ("hw_power_brake_slowdown", 0x80), ("display_clock_setting", 0x100))

    def __init__(self, gpu_uuid: str, period_s: float = 0.002):
        import threading
        self.sm, self.bits, self.mx, self.err = [], 0, None, None
        self.power_w = []
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml
            pynvml.nvmlInit()
            uuid = gpu_uuid if gpu_uuid.startswith("GPU-") else "GPU-" + gpu_uuid
            try:
                h = pynvml.nvmlDeviceGetHandleByUUID(uuid.encode())
            except Exception:
                h = pynvml.nvmlDeviceGetHandleByUUID(uuid)
            self.mx = float(pynvml.nvmlDeviceGetMaxClockInfo(h, pynvml.NVML_CLOCK_SM))
            reasons = getattr(pynvml, "nvmlDeviceGetCurrentClocksEventReasons", None) or \
                pynvml.nvmlDeviceGetCurrentClocksThrottleReasons

            def loop():
                while not self._stop.is_set():
                    try:
                        self.sm.append(float(pynvml.nvmlDeviceGetClockInfo(h, pynvml.NVML_CLOCK_SM)))
                        self.bits |= int(reasons(h))
                        self.power_w.append(pynvml.nvmlDeviceGetPowerUsage(h) / 1000.0)
                    except Exception as e:      # keep what was sampled
                        self.err = repr(e)
                        return
                    self._stop.wait(period_s)

            self._thread = threading.Thread(target=loop, daemon=True)
            self._thread.start()
        except Exception as e:
            self.err = repr(e)

    def stop(self) -> dict:
        if self._thread is not None:
            self._stop.set()
            self._thread.join(timeout=5)
        if not self.sm:
            return {"sm_mhz": None, "sm_max_mhz": self.mx, "reasons": ["no samples: " + str(self.err)]}
        return {"sm_mhz": statistics.median(self.sm), "sm_max_mhz": self.mx, "sm_mhz_min": min(self.sm),
                "reasons": [n for n, bit in self.REASONS if self.bits & bit], "reasons_mask": hex(self.bits),
                "power_w_max": max(self.power_w) if self.power_w else None, "samples": len(self.sm)}


def oracle_sample_run(d, n_seq):
    """Forward + backward of the float64 oracle on the first n_seq sequences; returns seconds."""
    from oracle import ssm_oracle as O
    done = None if d["done"] is None else d["done"][:n_seq]
    u, gy = d["u"][:n_seq], d["gy"][:n_seq]
    t0 = time.perf_counter()
    if "params" in d:      # stacked model
        _, cache = O.stack_fwd(d["params"], d["ln_weight"], d["ln_bias"], u, done)
        O.stack_bwd(d["params"], d["ln_weight"], d["ln_bias"], cache, done, gy)
        return time.perf_counter() - t0
    O.ssm_layer_fwd(d["Lambda"], d["Delta"], d["Bc"], d["Cc"], d["D"], u, done, None)
    O.ssm_layer_bwd(d["Lambda"], d["Delta"], d["Bc"], d["Cc"], d["D"], u, done, None, gy)
    return time.perf_counter() - t0


def blas_threads() -> int:
    try:
        from threadpoolctl import threadpool_info
        n = [p.get("num_threads", 1) for p in threadpool_info() if p.get("user_api") == "blas"]
        return max(n) if n else (os.cpu_count() or 1)
    except Exception:
        return os.cpu_count() or 1


def cpu_baseline(w, d, budget_s=15.0):
    """The oracle, as it stands, timed on a bounded sample of the workload's sequences."""
    have = d["u"].shape[0]
    n = min(have, 4)
    dt = oracle_sample_run(d, n)
    rate = n * w.T / dt
    n = int(max(1, min(have, budget_s * rate / w.T)))
    dt = oracle_sample_run(d, n)
    return {"value": n * w.T / dt, "unit": UNIT, "cores": blas_threads(), "kind": "oracle",
            "sample": f"first {n} of {w.B} sequences of {w.name} (T={w.T}, H={w.H}, P={w.P}), "
                      f"float64 forward+backward once, {dt:.1f} s"}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    w = I.WORKLOADS[args.workload]
    small = I.small_variant(w, B=min(w.B, max(1, 65536 // w.T)))
    d = I.draw_layer(small)
    n0 = min(small.B, 4)
    dt = oracle_sample_run(d, n0)
    per_step_budget = max(1.0, 120.0 / max(1, args.steps + args.warmup))
    n = int(max(1, min(small.B, per_step_budget * n0 / dt)))
    for _ in range(args.warmup):
        oracle_sample_run(d, n)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle_sample_run(d, n)
    total = time.perf_counter() - t0
    value = n * w.T * args.steps / total
    sample = f"first {n} sequences of {w.name} per step, float64 oracle forward+backward"
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * total / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": w.name, "B": w.B, "T": w.T, "H": w.H, "P": w.P, "io_dtype": w.io_dtype,
                   "sampled_sequences_per_step": n},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": blas_threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


def time_step_mode(w, torch, sb, n_traj=4096, steps=50):
    """Single-step mode (ssm_step) at the paper's imagination batch, 32 x 128 start states, with
    the workload's H, P and I/O type: a rollout of `steps` calls, the state updated in place,
    timed with CUDA events after a warm-up rollout.  Reported beside the headline, not part of it."""
    io = torch.bfloat16 if w.io_dtype == "bf16" else torch.float32
    d = I.draw_layer(I.small_variant(w, B=1, T=1, n_layers=1))
    shape = sb.make_shape(n_traj, 1, w.H, w.P, w.io_dtype)
    dev = lambda a, dt: torch.from_numpy(np.ascontiguousarray(a)).to(dt).cuda()
    ws = sb.alloc_workspace(sb.ssm_step_workspace_bytes(shape))
    sb.ssm_step_prepare(shape, dev(d["Lambda"], torch.complex64), dev(d["Delta"], torch.float32),
                        dev(d["Bc"], torch.complex64), dev(d["Cc"], torch.complex64), ws)
    D = dev(d["D"], torch.float32)
    g = torch.Generator(device="cuda")
    g.manual_seed(w.seed)
    u = torch.randn((steps, n_traj, w.H), device="cuda", generator=g).to(io)
    x = torch.zeros((n_traj, w.P), dtype=torch.complex64, device="cuda")
    y = torch.empty((n_traj, w.H), dtype=io, device="cuda")
    stream = torch.cuda.current_stream()
    for t in range(5):
        sb.ssm_step(shape, D, u[t], None, x, x, y, ws, stream)
    torch.cuda.synchronize()
    n0 = sb.ssm_launch_count()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for t in range(steps):
        sb.ssm_step(shape, D, u[t], None, x, x, y, ws, stream)
    e1.record(stream)
    torch.cuda.synchronize()
    sb.ssm_check(ws)
    eager_us = e0.elapsed_time(e1) * 1e3 / steps
    launches = (sb.ssm_launch_count() - n0) / steps
    # the same rollout captured once in a CUDA graph and replayed: no host work per step
    horizon = 15
    side = torch.cuda.Stream()
    side.wait_stream(stream)
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=side):
        for t in range(horizon):
            sb.ssm_step(shape, D, u[t], None, x, x, y, ws, side)
    torch.cuda.synchronize()
    graph.replay()
    torch.cuda.synchronize()
    g0, g1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    reps = 10
    g0.record()
    for _ in range(reps):
        graph.replay()
    g1.record()
    torch.cuda.synchronize()
    sb.ssm_check(ws)
    return {"trajectories": n_traj, "steps": steps, "us_per_step": eager_us, "launches_per_step": launches,
            "graph_horizon": horizon, "graph_us_per_step": g0.elapsed_time(g1) * 1e3 / (reps * horizon)}


def time_half_glu(w, torch, sb, steps=10):
    """The half-GLU gate (ssm_glu_fwd + ssm_glu_bwd) on the workload's [B, T, H] activations,
    device-resident, per-stage CUDA events.  Reported beside the headline, not part of it."""
    io = torch.bfloat16 if w.io_dtype == "bf16" else torch.float32
    shape = sb.make_shape(w.B, w.T, w.H, w.P, w.io_dtype)
    g = torch.Generator(device="cuda")
    g.manual_seed(w.seed + 1)
    W = (torch.randn((w.H, w.H), device="cuda", generator=g) / w.H ** 0.5).contiguous()
    v = torch.randn((w.B, w.T, w.H), device="cuda", generator=g).to(io)
    gout = torch.randn((w.B, w.T, w.H), device="cuda", generator=g).to(io)
    out, gv, dW = torch.empty_like(v), torch.empty_like(v), torch.empty_like(W)
    ws = sb.alloc_workspace(sb.ssm_glu_workspace_bytes(shape))
    stream = torch.cuda.current_stream()

    def step():
        sb.ssm_glu_fwd(shape, W, v, out, ws, stream)
        sb.ssm_glu_bwd(shape, W, v, gout, ws, gv, dW, stream)

    for _ in range(3):
        step()
    torch.cuda.synchronize()
    sb.ssm_profile_begin()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(steps):
        step()
    e1.record(stream)
    torch.cuda.synchronize()
    stages = sb.ssm_profile_end()
    sb.ssm_check(ws)
    ms = e0.elapsed_time(e1) / steps
    return {"ms_per_step": ms, "timesteps_per_sec": w.timesteps / (ms * 1e-3),
            "stage_ms_per_step": {k: round(v_[1] / steps, 4) for k, v_ in stages.items()}}


def time_workload(w, torch, sb, harness, steps=10, warmup=3, graph=False):
    """Forward + backward of one named workload with inputs drawn on the device: CUDA-event time per
    step, launches per step and the library's per-stage times.  With `graph` also the time of the step
    captured once in a CUDA graph and replayed (no host work per launch)."""
    d = harness.device_drawn(w)
    buf = harness.StackBuffers(d, w.io_dtype) if w.n_layers > 1 else harness.LayerBuffers(d, w.io_dtype)
    stream = torch.cuda.current_stream()
    for _ in range(warmup):
        buf.forward(stream)
        buf.backward(stream)
    torch.cuda.synchronize()
    sb.ssm_check(buf.ws)
    # A launch-bound step feels the library's per-stage events (two event records per stage: 32 x 128 at H = 512
    # takes 0.10 ms per step without them and 0.15 with), so small workloads are timed twice: first with nothing
    # between the kernels, then again with the stage events.  Large workloads (milliseconds per step, the events
    # cost under 1 %) are timed once, with the events, which keeps each of them a short burst like the headline:
    # after a few tens of milliseconds of back-to-back work the power cap lowers the SM clock (see "sustained").
    small = w.timesteps <= 32768
    n0 = sb.ssm_launch_count()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    if small:
        e0.record(stream)
        for _ in range(steps):
            buf.forward(stream)
            buf.backward(stream)
        e1.record(stream)
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1) / steps
    launches = (sb.ssm_launch_count() - n0) / steps if small else None
    n0 = sb.ssm_launch_count()
    sb.ssm_profile_begin()
    p0, p1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    p0.record(stream)
    for _ in range(steps):
        buf.forward(stream)
        buf.backward(stream)
    p1.record(stream)
    torch.cuda.synchronize()
    stages = sb.ssm_profile_end()
    if not small:
        ms = p0.elapsed_time(p1) / steps
        launches = (sb.ssm_launch_count() - n0) / steps
    out = {"B": w.B, "T": w.T, "H": w.H, "P": w.P, "io_dtype": w.io_dtype, "n_layers": w.n_layers,
           "ms_per_step": round(ms, 5), "timesteps_per_sec": w.timesteps / (ms * 1e-3),
           "launches_per_step": launches,
           "stage_events_in_timed_steps": not small, "ms_per_step_with_stage_events": round(p0.elapsed_time(p1) / steps, 5),
           "stage_ms_per_step": {k: round(v[1] / steps, 5) for k, v in stages.items()}}
    if graph:
        out["graph_ms_per_step"] = replay_ms(buf, torch, stream)
    sb.ssm_check(buf.ws)
    return out


def time_sustained(w, torch, harness, local, steps=300):
    """The headline workload for a few hundred back-to-back steps (about half a second): long enough for the
    power cap to settle the SM clock, which the 20-step timed region is not.  Reported beside the headline, not
    instead of it, with the clocks sampled meanwhile.  Runs last: what follows it would start power-capped."""
    buf = harness.LayerBuffers(harness.device_drawn(w), w.io_dtype)
    stream = torch.cuda.current_stream()
    for _ in range(3):
        buf.forward(stream)
        buf.backward(stream)
    torch.cuda.synchronize()
    sampler = ClockSampler(str(torch.cuda.get_device_properties(local).uuid))
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(steps):
        buf.forward(stream)
        buf.backward(stream)
    e1.record(stream)
    torch.cuda.synchronize()
    clocks = sampler.stop()
    ms = e0.elapsed_time(e1) / steps
    return {"steps": steps, "ms_per_step": round(ms, 5), "timesteps_per_sec": w.timesteps / (ms * 1e-3), "clocks": clocks}


def replay_ms(buf, torch, stream, reps=20):
    """A forward + backward captured once in a CUDA graph and replayed: milliseconds per replay."""
    side = torch.cuda.Stream()
    side.wait_stream(stream)
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g, stream=side):
        buf.forward(side)
        buf.backward(side)
    torch.cuda.synchronize()
    g.replay()
    torch.cuda.synchronize()
    g0, g1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    g0.record()
    for _ in range(reps):
        g.replay()
    g1.record()
    torch.cuda.synchronize()
    return round(g0.elapsed_time(g1) / reps, 5)


def time_paper_block(w, n_blocks, torch, sb, harness, steps=20):
    """The paper's sequence block (SSM layer, then the half-GLU gate on its output; Appendix "S5 Sequence
    Layer") n_blocks times in a row, forward + backward, at a workload's sizes: CUDA-event time per step,
    eager and replayed from a CUDA graph."""
    shape = sb.make_shape(w.B, w.T, w.H, w.P, w.io_dtype)
    layers = [harness.LayerBuffers(harness.device_drawn(I.small_variant(w, seed=w.seed + l)), w.io_dtype) for l in range(n_blocks)]
    g = torch.Generator(device="cuda")
    g.manual_seed(w.seed)
    Ws = [(torch.randn((w.H, w.H), device="cuda", generator=g) / w.H ** 0.5).contiguous() for _ in range(n_blocks)]
    dWs = [torch.empty_like(W) for W in Ws]
    gws = [sb.alloc_workspace(sb.ssm_glu_workspace_bytes(shape)) for _ in range(n_blocks)]
    outs = [torch.empty_like(layers[0].y) for _ in range(n_blocks)]
    gout = layers[0].gy.clone()
    for l, L in enumerate(layers):
        L.gy = torch.empty_like(L.y)
        if l > 0:
            L.u = outs[l - 1]

    def step(stream):
        for l, L in enumerate(layers):
            L.forward(stream)
            sb.ssm_glu_fwd(shape, Ws[l], L.y, outs[l], gws[l], stream)
        gr = gout
        for l in range(n_blocks - 1, -1, -1):
            L = layers[l]
            sb.ssm_glu_bwd(shape, Ws[l], L.y, gr, gws[l], L.gy, dWs[l], stream)
            L.backward(stream)
            gr = L.du

    stream = torch.cuda.current_stream()
    for _ in range(3):
        step(stream)
    torch.cuda.synchronize()
    n0 = sb.ssm_launch_count()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(steps):
        step(stream)
    e1.record(stream)
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / steps
    launches = (sb.ssm_launch_count() - n0) / steps

    class _Both:      # forward + backward of the chain, in the shape replay_ms wants
        def forward(self, s):
            step(s)

        def backward(self, s):
            pass

    out = {"blocks": n_blocks, "B": w.B, "T": w.T, "H": w.H, "P": w.P, "io_dtype": w.io_dtype,
           "ms_per_step": round(ms, 5), "timesteps_per_sec": w.timesteps / (ms * 1e-3), "launches_per_step": launches,
           "graph_ms_per_step": replay_ms(_Both(), torch, stream)}
    for L in layers:
        sb.ssm_check(L.ws)
    return out


def scan_stage_summary(r, peaks):
    """The two scan stages of a timed layer step (fused with their projections, or apart) as
    algorithmic GB/s and as fractions of the measured copy rate and of the nominal 8 TB/s."""
    s_io = 2 if r["io_dtype"] == "bf16" else 4
    n = r["B"] * r["T"]
    out = {}
    for key in ("gemm_Bu_scan_fwd", "scan_fwd", "gemm_gx_scan_bwd", "scan_bwd"):
        ms = r["stage_ms_per_step"].get(key)
        if ms:
            gbs = STAGE_MODEL[key][1](r["H"], r["P"], s_io) * n / (ms * 1e-3) / 1e9
            out[key] = {"ms": ms, "algorithmic_GBps": round(gbs, 1), "frac_of_measured_copy": round(gbs / peaks["hbm_gbs"], 4),
                        "frac_of_8TBps": round(gbs / 8000.0, 4)}
    return out


def time_scans_alone(T, torch, sb, peaks, P=256, rows=262144, steps=10):
    """ssm_scan_fwd / ssm_scan_bwd on their own (B * T = rows, fp32 complex states in and out):
    16 P bytes per timestep forward (Bu in, x out), 24 P backward (g_x and x in, s out)."""
    B = rows // T
    shape = sb.make_shape(B, T, 8, P, "f32")
    g = torch.Generator(device="cuda")
    g.manual_seed(T)
    cplx = lambda *s: torch.view_as_complex(torch.randn(s + (2,), device="cuda", generator=g))
    lam = -(0.01 + 0.99 * torch.rand(P, device="cuda", generator=g)) + 1j * 3.14159 * torch.rand(P, device="cuda", generator=g)
    dt = torch.exp(torch.log(torch.tensor(1e-3)) + torch.rand(P, device="cuda", generator=g) * torch.log(torch.tensor(100.0)))
    Abar = torch.exp(lam * dt).to(torch.complex64)
    Bu, gx = cplx(B, T, P), cplx(B, T, P)
    x, s = torch.empty_like(Bu), torch.empty_like(Bu)
    gA = torch.empty(P, dtype=torch.complex64, device="cuda")
    ws = sb.alloc_workspace(sb.ssm_scan_workspace_bytes(shape))
    stream = torch.cuda.current_stream()
    res = {"B": B, "T": T, "P": P}
    for name, call, bytes_per_ts in (
            ("ssm_scan_fwd", lambda: sb.ssm_scan_fwd(shape, Abar, Bu, None, None, x, None, ws, stream), 16.0 * P),
            ("ssm_scan_bwd", lambda: sb.ssm_scan_bwd(shape, Abar, None, None, x, gx, None, s, gA, None, ws, stream), 24.0 * P)):
        for _ in range(3):
            call()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(steps):
            call()
        e1.record(stream)
        torch.cuda.synchronize()
        sb.ssm_check(ws)
        ms = e0.elapsed_time(e1) / steps
        gbs = bytes_per_ts * rows / (ms * 1e-3) / 1e9
        res[name] = {"ms": round(ms, 5), "algorithmic_GBps": round(gbs, 1),
                     "frac_of_measured_copy": round(gbs / peaks["hbm_gbs"], 4), "frac_of_8TBps": round(gbs / 8000.0, 4)}
    return res


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD, choices=sorted(I.WORKLOADS))
    ap.add_argument("--impl", default="b200", choices=["b200", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--batch", type=int, default=0,
                    help="run the workload with this many sequences instead of its own B (cut-down cases for profiler "
                         "captures; the line says so and is not a headline number)")
    ap.add_argument("--scans-alone", type=int, default=0, metavar="T",
                    help="time only ssm_scan_fwd / ssm_scan_bwd at sequence length T (B*T = 262144 rows, or --batch "
                         "sequences) and print that (profiler captures of the stand-alone scan kernels)")
    ap.add_argument("--kernels-only", action="store_true",
                    help="stop after the device-resident timed steps and print their stage times only (profiler captures)")
    ap.add_argument("--no-extras", action="store_true",
                    help="skip the extra measurements reported beside the headline (sweep, scans alone, other configs)")
    ap.add_argument("--allreduce-grads", action="store_true",
                    help="N > 1: also sum the parameter gradients over the ranks every step (one all-reduce of the "
                         "gradient bucket, running under the next step's forward pass), as a data-parallel trainer would")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "b200" else args.warmup

    if args.impl == "reference":
        run_reference(args)
        return

    import torch
    import torch.distributed as dist
    from paper_2502_20168_b200 import binding as sb, harness

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device; there is no CPU fallback")
    torch.cuda.set_device(local)
    if world > 1:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))

    if args.scans_alone > 0:
        peaks, _ = load_peaks()
        T = args.scans_alone
        rows = args.batch * T if args.batch > 0 else 262144
        print(json.dumps({"scans_alone": time_scans_alone(T, torch, sb, peaks, rows=rows, steps=max(1, args.steps))}))
        return
    w = I.WORKLOADS[args.workload]
    if args.batch > 0:
        w = I.small_variant(w, B=args.batch)
    wr = I.small_variant(w, seed=w.seed + 1000 * rank)
    d = I.draw_layer(wr)
    stacked = w.n_layers > 1
    buf = harness.StackBuffers(d, w.io_dtype) if stacked else harness.LayerBuffers(d, w.io_dtype)
    stream = torch.cuda.current_stream()

    exchange = args.allreduce_grads and world > 1 and not stacked
    xchg = harness.GradExchange(buf) if exchange else None

    def step():
        buf.forward(stream)
        if xchg:                         # last step's gradient sum has to be out of the bucket before it is rewritten
            xchg.finish()
        buf.backward(stream)
        if xchg:
            xchg.start()

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(args.warmup):
        step()
    sb.ssm_check(buf.ws)
    barrier()

    # ---- timed region: device-resident inputs, per-stage events recorded by the library ----
    sampler = ClockSampler(str(torch.cuda.get_device_properties(local).uuid)) if rank == 0 else None
    launches0 = sb.ssm_launch_count()
    sb.ssm_profile_begin()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    ev0.record(stream)
    for _ in range(args.steps):
        step()
    if xchg:                             # the last step's exchange belongs to the timed region
        xchg.finish()
    ev1.record(stream)
    barrier()
    ms = ev0.elapsed_time(ev1)
    stages = sb.ssm_profile_end()
    launches = sb.ssm_launch_count() - launches0
    clocks = sampler.stop() if sampler else None
    sb.ssm_check(buf.ws)
    if args.kernels_only:
        if rank == 0:
            print(json.dumps({"kernels_only": True, "workload": w.name, "B": w.B, "T": w.T, "H": w.H, "P": w.P,
                              "steps": args.steps, "ms_per_step": ms / args.steps, "gpu_launches": int(launches),
                              "stage_ms_per_step": {k: round(v[1] / args.steps, 4) for k, v in stages.items()}}))
        if world > 1:
            dist.destroy_process_group()
        return

    # ---- end to end: pinned host inputs in, results out, every step ----
    in_names = ("u", "gout") if stacked else ("u", "gy")
    host_in = {k: getattr(buf, k).cpu().pin_memory() for k in in_names}
    if buf.done is not None:
        host_in["done"] = buf.done.cpu().pin_memory()
    out_names = ("out", "du") if stacked else ("y", "du", "dLambda", "dDelta", "dB", "dC", "dD")
    host_out = {k: torch.empty_like(getattr(buf, k), device="cpu").pin_memory() for k in out_names}
    h2d = sum(t.numel() * t.element_size() for t in host_in.values())
    d2h = sum(t.numel() * t.element_size() for t in host_out.values())

    e2e_steps = max(1, min(args.steps, 10))
    if stacked:
        def e2e_step():
            for k, t in host_in.items():
                getattr(buf, k).copy_(t, non_blocking=True)
            step()
            for k, t in host_out.items():
                t.copy_(getattr(buf, k), non_blocking=True)

        e2e_step()
        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(e2e_steps):
            e2e_step()
        e1.record(stream)
        barrier()
        e2e_ms = e0.elapsed_time(e1)
        e2e_mode = "copies and compute in sequence on one stream"
    else:
        # Every step still moves all of its inputs in and all of its results out; the copies of
        # neighbouring steps overlap the compute through two sets of input / output buffers and three
        # streams (in, compute, out), as a training loop that streams batches would do.
        s_in, s_out = torch.cuda.Stream(), torch.cuda.Stream()
        dev_in = [{k: torch.empty_like(getattr(buf, k)) for k in host_in} for _ in range(2)]
        dev_out = [{k: torch.empty_like(getattr(buf, k)) for k in host_out} for _ in range(2)]
        ev = lambda: torch.cuda.Event(enable_timing=True)
        in_done, comp_done, out_done = {}, {}, {}

        def pipeline(n):
            first, last = ev(), ev()
            first.record(stream)
            s_in.wait_event(first)
            for i in range(n):
                j = i % 2
                with torch.cuda.stream(s_in):
                    if i >= 2:
                        s_in.wait_event(comp_done[i - 2])      # step i-2 has consumed this input set
                    for k, t in host_in.items():
                        dev_in[j][k].copy_(t, non_blocking=True)
                    in_done[i] = ev()
                    in_done[i].record(s_in)
                stream.wait_event(in_done[i])
                if i >= 2:
                    stream.wait_event(out_done[i - 2])         # step i-2's results have left this output set
                for k, t in dev_in[j].items():
                    setattr(buf, k, t)
                for k, t in dev_out[j].items():
                    setattr(buf, k, t)
                step()
                comp_done[i] = ev()
                comp_done[i].record(stream)
                with torch.cuda.stream(s_out):
                    s_out.wait_event(comp_done[i])
                    for k, t in host_out.items():
                        t.copy_(dev_out[j][k], non_blocking=True)
                    out_done[i] = ev()
                    out_done[i].record(s_out)
            stream.wait_event(out_done[n - 1])
            last.record(stream)
            return first, last

        pipeline(2)
        barrier()
        e0, e1 = pipeline(e2e_steps)
        barrier()
        e2e_ms = e0.elapsed_time(e1)
        e2e_mode = "double-buffered: H2D, compute and D2H of neighbouring steps overlap on three streams"

    times = torch.tensor([ms, e2e_ms], dtype=torch.float64, device="cuda")
    if world > 1:
        dist.all_reduce(times, op=dist.ReduceOp.MAX)
    ms, e2e_ms = float(times[0]), float(times[1])

    if rank == 0:
        peaks, peak_kind = load_peaks()
        total_ts = w.timesteps * world
        value = total_ts * args.steps / (ms * 1e-3)
        s_io = 2 if w.io_dtype == "bf16" else 4
        top = max((k for k in stages if k in STAGE_MODEL), key=lambda k: stages[k][1])
        flops_fn, bytes_fn = STAGE_MODEL[top]
        n_launch, top_ms = stages[top]
        per_launch_s = top_ms * 1e-3 / n_launch
        traffic = NCU_TRAFFIC_PER_TIMESTEP.get(top) if (w.T, w.H, w.P, w.io_dtype, stacked) == (1024, 512, 256, "bf16", False) else None
        traffic = None if traffic is None else traffic * w.timesteps
        hbm_peak = float(peaks["hbm_gbs"])
        tensor_peak = float(peaks.get("bf16_tflops_sustained", peaks["bf16_tflops"]))
        alg_flops = flops_fn(w.H, w.P, s_io) * w.timesteps if flops_fn else 0.0
        alg_bytes = bytes_fn(w.H, w.P, s_io) * w.timesteps if bytes_fn else 0.0
        floors_s = {"tensor": alg_flops / (tensor_peak * 1e12), "hbm": alg_bytes / (hbm_peak * 1e9)}
        bound = max(floors_s, key=floors_s.get)
        if bound == "hbm":
            alg, achieved, peak, runit = alg_bytes, alg_bytes / per_launch_s / 1e9, hbm_peak, "GB/s"
        else:
            alg, achieved, peak, runit = alg_flops, alg_flops / per_launch_s / 1e12, tensor_peak, "TFLOP/s"
        stage_share = {k: round(v[1] / ms, 4) for k, v in stages.items()}
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms / args.steps, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None,
            "dtype": "bf16-io/bf16-hi+lo-mma/f32-acc+state" if w.io_dtype == "bf16" and not stacked else "f32",
            "data": "synthetic",
            "config": {"workload": w.name, "B": w.B, "T": w.T, "H": w.H, "P": w.P, "io_dtype": w.io_dtype,
                       "p_done": w.p_done, "n_layers": w.n_layers, "batch_override": args.batch > 0, "l2": "inputs larger than L2 (no flush)"
                       if w.timesteps * w.H * s_io > 126e6 else "inputs fit in L2", "parallelism": f"batch-sharded x{world}" + (" + gradient all-reduce" if exchange else "")},
            "e2e": {"value": total_ts * e2e_steps / (e2e_ms * 1e-3), "unit": UNIT, "h2d_bytes_per_step": h2d,
                    "d2h_bytes_per_step": d2h, "steps": e2e_steps, "mode": e2e_mode},
            "gpu_launches": int(launches),
            "clocks": clocks,
            "roofline": {"kernel": top, "bound": bound, "achieved": achieved, "peak": peak, "unit": runit,
                         "frac": achieved / peak, "traffic": traffic, "peak_source": peak_kind,
                         "frac_of_8TBps": (achieved / 8000.0) if bound == "hbm" else None,
                         "algorithmic_per_launch": alg,
                         "floor_ms": {k: round(v * 1e3, 4) for k, v in floors_s.items() if v > 0}, "launches_per_step": n_launch / args.steps,
                         "ms_per_launch": per_launch_s * 1e3},
            "stage_ms_per_step": {k: round(v[1] / args.steps, 4) for k, v in stages.items()},
            "stage_share": stage_share,
        }
        if world == 1 and not stacked:
            line["step_mode"] = time_step_mode(w, torch, sb)
            del buf
            torch.cuda.empty_cache()
            line["half_glu"] = time_half_glu(w, torch, sb)
        if world == 1 and not args.no_extras:
            # evidence beside the headline: the whole scan-scaling sweep, the scan entry points on their own,
            # and the other configurations (eager; the small ones also replayed from a CUDA graph)
            buf = None
            torch.cuda.empty_cache()
            sweep = {}
            for c in I.C4:
                r = time_workload(c, torch, sb, harness)
                sweep[c.name] = {"ms_per_step": r["ms_per_step"], "timesteps_per_sec": r["timesteps_per_sec"],
                                 "launches_per_step": r["launches_per_step"], "scan_stages": scan_stage_summary(r, peaks)}
                torch.cuda.empty_cache()
            line["sweep"] = sweep
            line["scan_alone"] = {f"T{t}": time_scans_alone(t, torch, sb, peaks) for t in (1024, 16384)}
            torch.cuda.empty_cache()
            line["configs"] = {c.name: time_workload(c, torch, sb, harness, steps=20, graph=True)
                               for c in (I.C0, I.C1, I.C2, I.C3, I.PAPER_STATE, I.PAPER_VISION)}
            # the paper's own blocks (layer + half-GLU gate): one at the state task's sizes, two at the vision task's
            line["paper_block"] = {"state": time_paper_block(I.PAPER_STATE, 1, torch, sb, harness),
                                   "vision": time_paper_block(I.PAPER_VISION, 2, torch, sb, harness)}
            if not stacked:
                torch.cuda.empty_cache()
                line["sustained"] = time_sustained(w, torch, harness, local)
        if world == 1 and not args.no_cpu_baseline:
            line["cpu_baseline"] = cpu_baseline(w, I.draw_layer(I.small_variant(w, B=min(w.B, max(1, 262144 // w.T)))))
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
