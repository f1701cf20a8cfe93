"""Seeded synthetic inputs for the S5 SSM layer (shapes of the paper's world-model batches).

This module only draws random numbers and casts them; it holds none of the
method's arithmetic, so both the CPU oracle's tests and the CUDA path can feed
from it without sharing any computation.

The paper trains its world model on replay batches of 32 x 128 steps with a
256/512-wide SSM state and a 512/1024-wide deterministic state (hyper-parameter
tables of the appendix); the synthetic tensors below have that structure:
  Re(Lambda) ~ U[-1, -0.01], Im(Lambda) ~ U[0, pi], log(Delta) ~ U[ln 1e-3, ln 1e-1],
  Re/Im of B and C ~ N(0, 1/H) each, D ~ N(0, 1), u ~ N(0, 1), gy ~ N(0, 1),
  done ~ Bernoulli(p_done) (episode boundaries are rare: O(1e-3..1e-2) per step).
Everything is drawn in float64 from numpy.random.default_rng(seed) in the fixed
order listed in `draw_layer`, cast ONCE to the storage precision (float32 for the
parameters, float32 or bfloat16 for u / gy), and those cast values are what every
consumer sees.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, replace

import numpy as np


@dataclass(frozen=True)
class Workload:
    name: str
    B: int
    T: int
    H: int
    P: int
    io_dtype: str = "f32"      # "f32" or "bf16": storage type of u, y, gy, du
    p_done: float = 0.0        # Bernoulli rate of the done flags (0 -> no flags)
    n_layers: int = 1
    seed: int = 0

    @property
    def timesteps(self) -> int:
        return self.B * self.T


# The five workloads the headline metric is quoted on.  C4 is a sweep at fixed B*T.
C0 = Workload("c0_tiny_fp32", B=1, T=64, H=32, P=16, io_dtype="f32", seed=0)
C1 = Workload("c1_wm_batch_fp32", B=16, T=64, H=256, P=128, io_dtype="f32", p_done=0.01, seed=1)
C2 = Workload("c2_stack4_bf16", B=16, T=64, H=512, P=256, io_dtype="bf16", p_done=0.01,
              n_layers=4, seed=2)
C3 = Workload("c3_long_bf16", B=16, T=1024, H=512, P=256, io_dtype="bf16", p_done=0.002, seed=3)
C4_TS = (64, 256, 1024, 4096, 16384)
C4 = tuple(Workload(f"c4_sweep_T{t}_bf16", B=262144 // t, T=t, H=512, P=256,
                    io_dtype="bf16", seed=4) for t in C4_TS)
# The paper's own training batch (32 sequences of 128 steps, hyper-parameter tables of the appendix):
# state task (deterministic state 512, SSM state 256) and vision task (1024 / 512).
PAPER_STATE = Workload("paper_state_batch_bf16", B=32, T=128, H=512, P=256, io_dtype="bf16", p_done=0.01, seed=5)
PAPER_VISION = Workload("paper_vision_batch_bf16", B=32, T=128, H=1024, P=512, io_dtype="bf16", p_done=0.01, seed=6)
WORKLOADS = {w.name: w for w in (C0, C1, C2, C3) + C4 + (PAPER_STATE, PAPER_VISION)}


def round_to_bf16(a: np.ndarray) -> np.ndarray:
    """Round float values to the nearest bfloat16 (ties to even); result is float32."""
    f = np.ascontiguousarray(a, dtype=np.float32)
    bits = f.view(np.uint32)
    lsb = (bits >> np.uint32(16)) & np.uint32(1)
    rounded = (bits + np.uint32(0x7FFF) + lsb) & np.uint32(0xFFFF0000)
    out = rounded.view(np.float32)
    nan = np.isnan(f)
    if nan.any():
        out = out.copy()
        out[nan] = np.nan
    return out.reshape(f.shape)


def cast_io(a: np.ndarray, io_dtype: str) -> np.ndarray:
    """Cast to the I/O storage precision; returned as float32 holding exact values."""
    if io_dtype == "f32":
        return np.ascontiguousarray(a, dtype=np.float32)
    if io_dtype == "bf16":
        return round_to_bf16(a)
    raise ValueError(f"unknown io dtype {io_dtype!r}")


def draw_params(rng: np.random.Generator, H: int, P: int) -> dict:
    """One layer's parameters, drawn in the order Lambda, Delta, B, C, D; stored in fp32."""
    re_l = rng.uniform(-1.0, -0.01, size=P)
    im_l = rng.uniform(0.0, math.pi, size=P)
    log_dt = rng.uniform(math.log(1e-3), math.log(1e-1), size=P)
    sd = 1.0 / math.sqrt(H)
    re_b = rng.normal(0.0, sd, size=(P, H))
    im_b = rng.normal(0.0, sd, size=(P, H))
    re_c = rng.normal(0.0, sd, size=(H, P))
    im_c = rng.normal(0.0, sd, size=(H, P))
    d = rng.normal(0.0, 1.0, size=H)
    return {
        "Lambda": (re_l + 1j * im_l).astype(np.complex64),
        "Delta": np.exp(log_dt).astype(np.float32),
        "Bc": (re_b + 1j * im_b).astype(np.complex64),
        "Cc": (re_c + 1j * im_c).astype(np.complex64),
        "D": d.astype(np.float32),
    }


def draw_layer(w: Workload, *, with_x0: bool = False, with_gxT: bool = False) -> dict:
    """All tensors of one workload.

    Order of draws: per layer (Lambda, Delta, B, C, D), then u, done, gy, and only if
    asked for, x0 and gxT (so the default stream of numbers never depends on them).
    For a stack, `params` is a list of per-layer dicts and `ln_weight`/`ln_bias` are
    the LayerNorm affine parameters at their initial values (1, 0).
    """
    rng = np.random.default_rng(w.seed)
    params = [draw_params(rng, w.H, w.P) for _ in range(w.n_layers)]
    u = cast_io(rng.normal(0.0, 1.0, size=(w.B, w.T, w.H)), w.io_dtype)
    if w.p_done > 0.0:
        done = (rng.random(size=(w.B, w.T)) < w.p_done).astype(np.uint8)
    else:
        done = None
    gy = cast_io(rng.normal(0.0, 1.0, size=(w.B, w.T, w.H)), w.io_dtype)
    out = {"workload": w, "u": u, "done": done, "gy": gy}
    if with_x0:
        out["x0"] = (rng.normal(size=(w.B, w.P)) + 1j * rng.normal(size=(w.B, w.P))).astype(np.complex64)
    if with_gxT:
        out["gxT"] = (rng.normal(size=(w.B, w.P)) + 1j * rng.normal(size=(w.B, w.P))).astype(np.complex64)
    if w.n_layers == 1:
        out.update(params[0])
    else:
        out["params"] = params
        out["ln_weight"] = [np.ones(w.H, np.float32) for _ in range(w.n_layers)]
        out["ln_bias"] = [np.zeros(w.H, np.float32) for _ in range(w.n_layers)]
    return out


def draw_glu(w: Workload) -> dict:
    """Inputs of the half-GLU gate at a workload's B, T, H: weights W ~ N(0, 1/H) (fp32), the gate's
    input v ~ N(0, 1) (it stands in for the SSM output) and the output gradient gout ~ N(0, 1),
    both in the workload's I/O precision.  Its own stream of numbers (seed + 7919)."""
    rng = np.random.default_rng(w.seed + 7919)
    W = rng.normal(0.0, 1.0 / math.sqrt(w.H), size=(w.H, w.H)).astype(np.float32)
    v = cast_io(rng.normal(size=(w.B, w.T, w.H)), w.io_dtype)
    gout = cast_io(rng.normal(size=(w.B, w.T, w.H)), w.io_dtype)
    return {"W": W, "v": v, "gout": gout}


def small_variant(w: Workload, **changes) -> Workload:
    """Same distributions, other sizes (used by edge-case tests)."""
    return replace(w, **changes)


def shard_batch(B: int, rank: int, world: int) -> tuple[int, int]:
    """Contiguous [lo, hi) slice of the batch owned by `rank` (sequences are independent)."""
    base, rem = divmod(B, world)
    lo = rank * base + min(rank, rem)
    return lo, lo + base + (1 if rank < rem else 0)
