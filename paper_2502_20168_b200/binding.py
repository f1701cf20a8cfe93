"""Thin ctypes binding of libssm_b200.so: argument marshalling only.

Every function has the name and argument order of its C entry point in
include/ssm.h and takes torch CUDA tensors (used purely as device buffers) or
None for optional pointers.  Nothing is computed here; if the library is
missing or a call fails this raises, there is no other code path.
"""
from __future__ import annotations

import ctypes
import os
from ctypes import POINTER, Structure, byref, c_char_p, c_int, c_int32, c_size_t, c_void_p

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libssm_b200.so")

SSM_F32, SSM_BF16 = 0, 1
SSM_OK = 0
SSM_ERR_NULL, SSM_ERR_SHAPE, SSM_ERR_ALIGN, SSM_ERR_DTYPE = -1, -2, -3, -4
SSM_ERR_WORKSPACE, SSM_ERR_CUDA, SSM_ERR_TIMEOUT = -5, -6, -7

EXPORTS = (
    "ssm_status_string", "ssm_check", "ssm_discretize", "ssm_discretize_bwd",
    "ssm_scan_workspace_bytes", "ssm_scan_fwd", "ssm_scan_bwd",
    "ssm_layer_workspace_bytes", "ssm_layer_plan_string", "ssm_layer_fwd", "ssm_layer_bwd",
    "ssm_launch_count", "ssm_profile_begin", "ssm_profile_end", "ssm_scan_bwd_static", "ssm_check_static",
    "ssm_stack_workspace_bytes", "ssm_stack_fwd", "ssm_stack_bwd",
    "ssm_step_workspace_bytes", "ssm_step_prepare", "ssm_step",
    "ssm_glu_workspace_bytes", "ssm_glu_fwd", "ssm_glu_bwd",
)
SSM_ERR_TOO_LARGE = -8
SSM_STATIC_SCRATCH_BYTES = 8 << 20


class ssm_shape(Structure):
    _fields_ = [("B", c_int32), ("T", c_int32), ("H", c_int32), ("P", c_int32),
                ("io_dtype", c_int32), ("reserved", c_int32)]


class ssm_stack_params(Structure):
    _fields_ = [(n, c_void_p) for n in ("Lambda", "Delta", "Bc", "Cc", "D", "ln_weight", "ln_bias")]


class ssm_stack_grads(Structure):
    _fields_ = [(n, c_void_p) for n in ("dLambda", "dDelta", "dB", "dC", "dD", "dln_weight", "dln_bias")]


class SsmError(RuntimeError):
    def __init__(self, code: int, what: str):
        super().__init__(f"{what}: {status_string(code)} ({code})")
        self.code = code


def _load() -> ctypes.CDLL:
    if not os.path.exists(LIB_PATH):
        raise ImportError(
            f"{LIB_PATH} not found: build it with `python -m paper_2502_20168_b200.build` "
            "(there is no fallback implementation)")
    lib = ctypes.CDLL(LIB_PATH)
    P = c_void_p
    S = POINTER(ssm_shape)
    lib.ssm_status_string.restype = c_char_p
    lib.ssm_status_string.argtypes = [c_int]
    lib.ssm_check.restype = c_int
    lib.ssm_check.argtypes = [P, P]
    lib.ssm_discretize.restype = c_int
    lib.ssm_discretize.argtypes = [S] + [P] * 6
    lib.ssm_discretize_bwd.restype = c_int
    lib.ssm_discretize_bwd.argtypes = [S] + [P] * 9
    lib.ssm_scan_workspace_bytes.restype = c_size_t
    lib.ssm_scan_workspace_bytes.argtypes = [S]
    lib.ssm_scan_fwd.restype = c_int
    lib.ssm_scan_fwd.argtypes = [S] + [P] * 7 + [c_size_t, P]
    lib.ssm_scan_bwd.restype = c_int
    lib.ssm_scan_bwd.argtypes = [S] + [P] * 10 + [c_size_t, P]
    lib.ssm_layer_workspace_bytes.restype = c_size_t
    lib.ssm_layer_workspace_bytes.argtypes = [S]
    lib.ssm_layer_plan_string.restype = c_int
    lib.ssm_layer_plan_string.argtypes = [S, ctypes.c_char_p, c_size_t]
    lib.ssm_layer_fwd.restype = c_int
    lib.ssm_layer_fwd.argtypes = [S] + [P] * 11 + [c_size_t, P]
    lib.ssm_layer_bwd.restype = c_int
    lib.ssm_layer_bwd.argtypes = [S] + [P] * 11 + [c_size_t] + [P] * 8
    lib.ssm_scan_bwd_static.restype = c_int
    lib.ssm_scan_bwd_static.argtypes = [S] + [P] * 10
    lib.ssm_check_static.restype = c_int
    lib.ssm_check_static.argtypes = [P]
    lib.ssm_stack_workspace_bytes.restype = c_size_t
    lib.ssm_stack_workspace_bytes.argtypes = [S, c_int]
    lib.ssm_stack_fwd.restype = c_int
    lib.ssm_stack_fwd.argtypes = [S, c_int, POINTER(ssm_stack_params), P, P, P, P, c_size_t, P]
    lib.ssm_stack_bwd.restype = c_int
    lib.ssm_stack_bwd.argtypes = [S, c_int, POINTER(ssm_stack_params), P, P, P, P, c_size_t, P,
                                  POINTER(ssm_stack_grads), P]
    lib.ssm_step_workspace_bytes.restype = c_size_t
    lib.ssm_step_workspace_bytes.argtypes = [S]
    lib.ssm_step_prepare.restype = c_int
    lib.ssm_step_prepare.argtypes = [S] + [P] * 5 + [c_size_t, P]
    lib.ssm_step.restype = c_int
    lib.ssm_step.argtypes = [S] + [P] * 7 + [c_size_t, P]
    lib.ssm_glu_workspace_bytes.restype = c_size_t
    lib.ssm_glu_workspace_bytes.argtypes = [S]
    lib.ssm_glu_fwd.restype = c_int
    lib.ssm_glu_fwd.argtypes = [S] + [P] * 4 + [c_size_t, P]
    lib.ssm_glu_bwd.restype = c_int
    lib.ssm_glu_bwd.argtypes = [S] + [P] * 4 + [c_size_t] + [P] * 3
    lib.ssm_launch_count.restype = ctypes.c_longlong
    lib.ssm_launch_count.argtypes = []
    lib.ssm_profile_begin.restype = c_int
    lib.ssm_profile_begin.argtypes = []
    lib.ssm_profile_end.restype = c_int
    lib.ssm_profile_end.argtypes = [ctypes.c_char_p, c_size_t]
    return lib


_lib = _load()


def lib() -> ctypes.CDLL:
    return _lib


def status_string(code: int) -> str:
    return _lib.ssm_status_string(int(code)).decode()


def make_shape(B: int, T: int, H: int, P: int, io_dtype) -> ssm_shape:
    if isinstance(io_dtype, torch.dtype):
        io_dtype = {torch.float32: SSM_F32, torch.bfloat16: SSM_BF16}[io_dtype]
    elif isinstance(io_dtype, str):
        io_dtype = {"f32": SSM_F32, "bf16": SSM_BF16}[io_dtype]
    return ssm_shape(B, T, H, P, int(io_dtype), 0)


def _ptr(t):
    if t is None:
        return c_void_p(0)
    if isinstance(t, int):
        return c_void_p(t)
    if not t.is_cuda:
        raise ValueError("expected a CUDA tensor")
    if not t.is_contiguous():
        raise ValueError("expected a contiguous tensor")
    return c_void_p(t.data_ptr())


def _stream(stream=None):
    s = torch.cuda.current_stream() if stream is None else stream
    return c_void_p(s.cuda_stream)


def _nbytes(t) -> int:
    return 0 if t is None else t.numel() * t.element_size()


def _ok(code: int, what: str) -> None:
    if code != SSM_OK:
        raise SsmError(code, what)


def ssm_check(ws, stream=None) -> None:
    _ok(_lib.ssm_check(_ptr(ws), _stream(stream)), "ssm_check")


def ssm_discretize(shape, Lambda, Delta, Bc, Abar, Bbar, stream=None) -> None:
    _ok(_lib.ssm_discretize(byref(shape), _ptr(Lambda), _ptr(Delta), _ptr(Bc), _ptr(Abar), _ptr(Bbar),
                            _stream(stream)), "ssm_discretize")


def ssm_discretize_bwd(shape, Lambda, Delta, Bc, gAbar, gBbar, dLambda, dDelta, dB, stream=None) -> None:
    _ok(_lib.ssm_discretize_bwd(byref(shape), _ptr(Lambda), _ptr(Delta), _ptr(Bc), _ptr(gAbar), _ptr(gBbar),
                                _ptr(dLambda), _ptr(dDelta), _ptr(dB), _stream(stream)), "ssm_discretize_bwd")


def ssm_scan_workspace_bytes(shape) -> int:
    return int(_lib.ssm_scan_workspace_bytes(byref(shape)))


def ssm_scan_fwd(shape, Abar, Bu, done, x0, x, xT, ws, stream=None) -> None:
    _ok(_lib.ssm_scan_fwd(byref(shape), _ptr(Abar), _ptr(Bu), _ptr(done), _ptr(x0), _ptr(x), _ptr(xT),
                          _ptr(ws), _nbytes(ws), _stream(stream)), "ssm_scan_fwd")


def ssm_scan_bwd(shape, Abar, done, x0, x, gx, gxT, gBu, gAbar, gx0, ws, stream=None) -> None:
    _ok(_lib.ssm_scan_bwd(byref(shape), _ptr(Abar), _ptr(done), _ptr(x0), _ptr(x), _ptr(gx), _ptr(gxT),
                          _ptr(gBu), _ptr(gAbar), _ptr(gx0), _ptr(ws), _nbytes(ws), _stream(stream)),
        "ssm_scan_bwd")


def ssm_scan_bwd_static(shape, Abar, done, x0, x, gx, gxT, gBu, gAbar, gx0, stream=None) -> None:
    """ssm_scan_bwd for callers that cannot allocate a workspace: the library's own fixed
    scratch array is used instead (shared by all calls on the device, so do not overlap them;
    raises SsmError(SSM_ERR_TOO_LARGE) when the shape needs more than SSM_STATIC_SCRATCH_BYTES)."""
    _ok(_lib.ssm_scan_bwd_static(byref(shape), _ptr(Abar), _ptr(done), _ptr(x0), _ptr(x), _ptr(gx), _ptr(gxT),
                                 _ptr(gBu), _ptr(gAbar), _ptr(gx0), _stream(stream)), "ssm_scan_bwd_static")


def ssm_check_static(stream=None) -> None:
    """Status of the most recent ssm_scan_bwd_static call on the current device (synchronises `stream`)."""
    _ok(_lib.ssm_check_static(_stream(stream)), "ssm_check_static")


def ssm_layer_workspace_bytes(shape) -> int:
    return int(_lib.ssm_layer_workspace_bytes(byref(shape)))


def ssm_layer_plan_string(shape) -> str:
    buf = ctypes.create_string_buffer(160)
    _ok(_lib.ssm_layer_plan_string(byref(shape), buf, len(buf)), "ssm_layer_plan_string")
    return buf.value.decode()


def ssm_layer_fwd(shape, Lambda, Delta, Bc, Cc, D, u, done, x0, y, xT, ws, stream=None) -> None:
    _ok(_lib.ssm_layer_fwd(byref(shape), _ptr(Lambda), _ptr(Delta), _ptr(Bc), _ptr(Cc), _ptr(D), _ptr(u),
                           _ptr(done), _ptr(x0), _ptr(y), _ptr(xT), _ptr(ws), _nbytes(ws), _stream(stream)),
        "ssm_layer_fwd")


def ssm_layer_bwd(shape, Lambda, Delta, Bc, Cc, D, u, done, x0, gy, gxT, ws, du, dLambda, dDelta, dB, dC, dD,
                  dx0, stream=None) -> None:
    _ok(_lib.ssm_layer_bwd(byref(shape), _ptr(Lambda), _ptr(Delta), _ptr(Bc), _ptr(Cc), _ptr(D), _ptr(u),
                           _ptr(done), _ptr(x0), _ptr(gy), _ptr(gxT), _ptr(ws), _nbytes(ws), _ptr(du),
                           _ptr(dLambda), _ptr(dDelta), _ptr(dB), _ptr(dC), _ptr(dD), _ptr(dx0),
                           _stream(stream)), "ssm_layer_bwd")


def ssm_step_workspace_bytes(shape) -> int:
    return int(_lib.ssm_step_workspace_bytes(byref(shape)))


def ssm_step_prepare(shape, Lambda, Delta, Bc, Cc, ws, stream=None) -> None:
    _ok(_lib.ssm_step_prepare(byref(shape), _ptr(Lambda), _ptr(Delta), _ptr(Bc), _ptr(Cc), _ptr(ws), _nbytes(ws),
                              _stream(stream)), "ssm_step_prepare")


def ssm_step(shape, D, u, done, x_prev, x_next, y, ws, stream=None) -> None:
    _ok(_lib.ssm_step(byref(shape), _ptr(D), _ptr(u), _ptr(done), _ptr(x_prev), _ptr(x_next), _ptr(y), _ptr(ws),
                      _nbytes(ws), _stream(stream)), "ssm_step")


def ssm_glu_workspace_bytes(shape) -> int:
    return int(_lib.ssm_glu_workspace_bytes(byref(shape)))


def ssm_glu_fwd(shape, W, v, out, ws, stream=None) -> None:
    _ok(_lib.ssm_glu_fwd(byref(shape), _ptr(W), _ptr(v), _ptr(out), _ptr(ws), _nbytes(ws), _stream(stream)),
        "ssm_glu_fwd")


def ssm_glu_bwd(shape, W, v, gout, ws, gv, dW, stream=None) -> None:
    _ok(_lib.ssm_glu_bwd(byref(shape), _ptr(W), _ptr(v), _ptr(gout), _ptr(ws), _nbytes(ws), _ptr(gv), _ptr(dW),
                         _stream(stream)), "ssm_glu_bwd")


def _struct_array(cls, dicts):
    """Host array of structs of device pointers, one per layer (dicts of name -> tensor)."""
    arr = (cls * len(dicts))()
    for i, d in enumerate(dicts):
        for name, _ in cls._fields_:
            setattr(arr[i], name, _ptr(d[name]).value)
    return arr


def ssm_stack_workspace_bytes(shape, n_layers: int) -> int:
    return int(_lib.ssm_stack_workspace_bytes(byref(shape), int(n_layers)))


def ssm_stack_fwd(shape, params, u, done, out, ws, stream=None) -> None:
    """params: list (one per layer) of dicts Lambda, Delta, Bc, Cc, D, ln_weight, ln_bias of tensors."""
    arr = _struct_array(ssm_stack_params, params)
    _ok(_lib.ssm_stack_fwd(byref(shape), len(params), arr, _ptr(u), _ptr(done), _ptr(out), _ptr(ws), _nbytes(ws),
                           _stream(stream)), "ssm_stack_fwd")


def ssm_stack_bwd(shape, params, u, done, gout, ws, du, grads, stream=None) -> None:
    """grads: list of dicts dLambda, dDelta, dB, dC, dD, dln_weight, dln_bias of output tensors."""
    arr = _struct_array(ssm_stack_params, params)
    garr = _struct_array(ssm_stack_grads, grads)
    _ok(_lib.ssm_stack_bwd(byref(shape), len(params), arr, _ptr(u), _ptr(done), _ptr(gout), _ptr(ws), _nbytes(ws),
                           _ptr(du), garr, _stream(stream)), "ssm_stack_bwd")


def ssm_launch_count() -> int:
    return int(_lib.ssm_launch_count())


def ssm_profile_begin() -> None:
    _ok(_lib.ssm_profile_begin(), "ssm_profile_begin")


def ssm_profile_end() -> dict:
    """Stage name -> (launches, total milliseconds) recorded since ssm_profile_begin."""
    buf = ctypes.create_string_buffer(1 << 16)
    _ok(_lib.ssm_profile_end(buf, len(buf)), "ssm_profile_end")
    out = {}
    for line in buf.value.decode().splitlines():
        name, count, ms = line.split()
        out[name] = (int(count), float(ms))
    return out


def alloc_workspace(nbytes: int, device="cuda") -> torch.Tensor:
    """A 256-byte aligned device buffer (torch's caching allocator aligns to 512)."""
    return torch.empty(max(int(nbytes), 256), dtype=torch.uint8, device=device)
