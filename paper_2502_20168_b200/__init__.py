"""B200 (sm_100a) implementation of the S5 state-space layer of arxiv 2502.20168.

`inputs` draws the seeded synthetic workloads; `binding` is the ctypes layer over the
CUDA library (imported on first use, raises if the library has not been built);
`harness` moves numpy tensors to the device and calls the binding.
"""
from . import inputs  # noqa: F401

__all__ = ["inputs", "binding", "harness", "build"]


def __getattr__(name):
    if name in ("binding", "harness", "build"):
        import importlib
        return importlib.import_module(f"{__name__}.{name}")
    raise AttributeError(name)
